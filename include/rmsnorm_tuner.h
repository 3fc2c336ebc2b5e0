/*
 * rmsnorm_tuner.h - C ABI of the template-plus-search tuner for the fused
 * residual-add + RMSNorm kernel on sm_100a (NVIDIA B200).
 *
 * The library holds three things, after the paper's Level 2 ("parameter search
 * within the resource-feasible region", Algorithm 1) applied to one of its three
 * evaluation kernels, `fused_add_rmsnorm` ("Kernels" paragraph, Experimental
 * Setup):
 *
 *   1. the kernel as an explicitly parameterised template  (Templatize /
 *      Instantiate(S~, theta), Section "Problem Formulation" and Algorithm 1);
 *   2. the feasible-region deriver  (DeriveFeasibleSpace(S~, h, r(h)), Algorithm 1
 *      and Section "Tuning parameter selection and search space derivation");
 *   3. the guided search on measured device time with a correctness gate on every
 *      candidate  (Search(S~, x, Theta_feasible), Algorithm 1; timing protocol of
 *      "Performance Measurement": 20 warm-up runs then the mean of 100 runs;
 *      correctness as in paragraph "Correctness": max_i d(S~(x_i), S(x_i)) <= eps).
 *
 * The operator, per token row t (rows are independent):
 *     s_j  = fp32(x[t,j]) + fp32(r[t,j])               (one binary32 addition)
 *     r_out[t,j] = round_to_nearest_even_dtype(s_j)
 *     y[t,j] = round_dtype( s_j * rsqrt(mean_j(s_j^2) + eps) * w[j] )
 * The normalisation uses the un-rounded fp32 sum s_j.
 *
 * Conventions
 *   - Every function returns an rt_status (0 = RT_OK) unless stated; none throws,
 *     aborts or exits.  rt_last_error() gives the text of the last failure on the
 *     calling thread.
 *   - "device" pointers are CUDA global-memory addresses on the current device;
 *     "host" pointers are ordinary process memory.  The caller owns every buffer
 *     it passes; the library never frees or keeps them.
 *   - Tensors are row-major and contiguous: x, r, y, r_out are [n_tokens, hidden]
 *     with row stride `hidden` elements; w is [hidden]; all of element type
 *     `dtype`.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *   - Nothing here synchronises the device unless its comment says so.
 */
#ifndef RMSNORM_TUNER_H_
#define RMSNORM_TUNER_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { RT_BF16 = 0, RT_FP16 = 1, RT_FP32 = 2 } rt_dtype;

/* Most partial inputs and most destinations one launch of the all-reduce-fused norm takes. */
#define RT_MAX_PARTS 8

/* The kernels that have a template in this library (the paper tunes three serving kernels, "Kernels"). */
typedef enum {
    RT_OP_ADD_RMSNORM = 0,  /* fused residual-add + RMSNorm: the operator described above */
    RT_OP_SILU_AND_MUL = 1, /* out[t,j] = silu(x[t,j]) * x[t,d+j] for x of shape [n_tokens, 2*d] */
    RT_OP_MERGE_ATTN_STATES = 2, /* two partial attention results merged by their log-sum-exps */
    RT_OP_ADD_RMSNORM_FP8 = 3,   /* add_rmsnorm whose y leaves as e4m3 bytes with one scale per token */
    RT_OP_ADD_RMSNORM_ALLREDUCE = 4 /* add_rmsnorm whose x arrives as n_parts partial results (one per rank of a
                                       tensor-parallel group) that are summed while they are loaded */
} rt_op;

/* Where a row lives between the two passes over it. */
typedef enum {
    RT_STAGE_REG = 0,      /* ld.global vectors straight into registers, row kept as fp32 registers */
    RT_STAGE_SMEM_LDG = 1, /* ld.global vectors, sum kept as fp32 in shared memory */
    RT_STAGE_SMEM_TMA = 2, /* cp.async.bulk (TMA, one copy per row slice) into shared memory + mbarrier */
    RT_STAGE_REG_REALIGN = 3, /* add_rmsnorm only, for rows whose byte length is not a multiple of the vector width
                                (the paper's "vectorization and alignment strategies" axis): the row is cut at the
                                vec_bytes boundaries of the tensor; the whole chunks between them move as vectors of
                                vec_bytes and stay in registers, the fewer than vec_bytes bytes before the first and
                                after the last boundary move one element to a thread.  Takes vec_bytes = 16 or 32, the
                                shuffle reduction, base pointers aligned to vec_bytes and any hidden size */
    RT_STAGE_TMA_PIPELINE = 4 /* add_rmsnorm only ("loop scheduling" in the paper's list of tuning dimensions): a
                                 persistent grid - as many CTAs as stay resident on the device, each walking over row
                                 blocks b, b + grid, ... - with a ring of `unroll` shared-memory stages per row slot
                                 (1, 2 or 4), so that the TMA bulk copies of the CTA's next `unroll` - 1 row blocks
                                 are in flight while the current one is reduced and stored.  Same alignment rules as
                                 RT_STAGE_SMEM_TMA; shuffle or shared-memory reduction, no cluster.  Left out of the
                                 derived feasible set unless RT_PRUNE_PIPELINE_STAGE is cleared from the mask */
} rt_stage;

/* How the per-row sum of squares is combined. */
typedef enum {
    RT_REDUCE_SHFL = 0,   /* warp shuffle tree, then one shared-memory hop across warps */
    RT_REDUCE_SMEM = 1,   /* shared-memory halving tree over all threads of the row */
    RT_REDUCE_CLUSTER = 2 /* a row is split over a thread-block cluster; partials meet through
                             distributed shared memory and barrier.cluster */
} rt_reduce;

/* theta: one point of the template's parameter space. */
typedef struct {
    int32_t threads_per_row; /* threads cooperating on one row (blockDim.x); power of two, 32..1024 */
    int32_t rows_per_cta;    /* rows handled by one CTA (blockDim.y); 1..8 */
    int32_t vec_bytes;       /* bytes per ld/st: 32 (the 256-bit global accesses of sm_100), 16
                                or 8 (4 and 2 exist as a narrow fall-back); 16 or 32 with
                                RT_STAGE_REG_REALIGN, whatever the row length */
    int32_t unroll;          /* independent vector loads in flight per thread and tensor: 1, 2, 4 */
    int32_t stage;           /* rt_stage */
    int32_t reduce;          /* rt_reduce */
    int32_t cluster_size;    /* CTAs per row when reduce == RT_REDUCE_CLUSTER (2, 4, 8), else 1 */
} rt_params;

typedef struct {
    int64_t n_tokens;
    int64_t hidden;        /* row width of the OUTPUT: hidden size; d for silu_and_mul; heads * d for
                              merge_attn_states */
    int32_t dtype;         /* rt_dtype */
    int32_t min_ptr_align; /* largest power of two (bytes, <= 256) dividing all base addresses */
    int32_t op;            /* rt_op; 0 = add_rmsnorm */
    int32_t head_dim;      /* merge_attn_states: d (hidden = heads * d); 0 for the other kernels */
    int32_t n_parts;       /* all-reduce-fused norm: partial inputs summed per element (2, 4 or 8); 0 otherwise */
    int32_t reserved;      /* 0 */
} rt_shape;

/* r(h): the resource upper bounds the feasible region is derived from. */
typedef struct {
    int32_t sm_count;
    int32_t warp_size;
    int32_t max_threads_per_block;
    int32_t max_threads_per_sm;
    int32_t max_blocks_per_sm;
    int32_t regs_per_block;
    int32_t regs_per_sm;
    int32_t max_regs_per_thread;
    int32_t max_cluster_size;
    int32_t have_device;            /* 1: per-kernel registers/spills and occupancy come from the CUDA
                                       runtime; 0: registers, spills and shared memory come from the
                                       compiler's report for the library as compiled, occupancy from arithmetic on r(h) */
    int64_t smem_per_block_optin;   /* largest dynamic + static shared memory one CTA may ask for */
    int64_t smem_per_sm;
    int64_t smem_reserved_per_block;
    int64_t l2_bytes;
} rt_limits;

/* Heuristic ("obvious inefficiency") pruning rules; hard rules are always applied. */
enum {
    RT_PRUNE_IDLE_THREADS = 1,  /* half the threads of the row or more would never own a vector */
    RT_PRUNE_DUPLICATES = 2,    /* unroll deeper than the per-thread vector count: same kernel again */
    RT_PRUNE_CLUSTER_WAVES = 4, /* split rows over a cluster only while whole rows cannot fill the SMs */
    RT_PRUNE_IDLE_ROWS = 8,     /* more rows per CTA than the batch has rows */
    RT_PRUNE_PIPELINE_STAGE = 16, /* RT_STAGE_TMA_PIPELINE: measured on B200 it wins on no shape tried, so the
                                     default search does not pay for its points; clear the bit to include them */
    RT_PRUNE_BYTES_IN_FLIGHT = 32, /* Little's law on the loads.  On a batch of two waves of CTAs or more: theta keeps
                                      fewer than 32 KB of input in flight per SM (resident CTAs x what one CTA requests
                                      before it consumes anything: a row slice per input in the bulk-copy stages, one
                                      batch of `unroll` vectors per thread and input otherwise) while some other theta
                                      of the shape reaches that.  B200 needs 16-22 KB per SM (3.3 TB/s of reads x
                                      0.7-1 us); of 7579 such points timed in 59 exhaustive sweeps none came within
                                      21 % of its shape's optimum.  Not applied to the fall-back vector widths (4, 2
                                      bytes) nor to merge_attn_states */
    RT_PRUNE_DEFAULT = 63
};

typedef enum { RT_SEARCH_GUIDED = 0, RT_SEARCH_EXHAUSTIVE = 1 } rt_strategy;

typedef struct {
    int32_t max_evals;       /* budget in kernel evaluations (one evaluation = gate + warm-up + timed runs) */
    int32_t warmup;          /* untimed launches per evaluation (paper: 20) */
    int32_t iters;           /* timed launches per block (paper: 100); time = block time / iters */
    int32_t repeats;         /* timed blocks per evaluation; the score is their median (>= 1) */
    int32_t top_k;           /* finalists re-timed before the winner is declared (0 = none) */
    int32_t strategy;        /* rt_strategy */
    int32_t heuristics;      /* RT_PRUNE_* mask used for the candidate set */
    int32_t use_graph;       /* 1: the timed block is one CUDA graph of `iters` launches */
    const rt_params* seeds;  /* host; evaluated first when given (configs found on other shapes) */
    int32_t n_seeds;
    int32_t preheat_ms;      /* 0..5000: before its first timing, and again before the Top-K re-test (and at the start
                                of tuner_retest_interleaved), the tuner keeps the device busy for this long with
                                launches of a candidate that has passed its gate, so that candidates are compared at
                                the clocks of a loaded device instead of at the boost clocks of one that was waiting
                                for the host.  0 = no pre-heating */
} rt_budget;

/* For silu_and_mul: x is the [n_tokens, 2*d] input (ring stride 2 * ring_stride_bytes), y the output,
 * y_ref its reference; r, w, r_out, r_ref are unused and may be NULL.
 * For merge_attn_states: x = v_a, r = v_b, w = s_a, aux = s_b, y = v_out, r_out = s_out, y_ref and r_ref their
 * references (the s tensors are binary32 [n_tokens, heads]; in a ring they advance by n_tokens*heads*4).
 * For the fp8-output norm: y = q (bytes, ring stride ring_stride_bytes / 2), y_ref its reference codes,
 * aux_out = scale ([n_tokens] binary32, ring stride n_tokens*4), aux_ref its reference.
 * For the all-reduce-fused norm: x holds the n_parts partial inputs one after the other, part k at byte offset
 * k * n_tokens * hidden * sizeof(element) (ring stride n_parts * ring_stride_bytes); everything else as for
 * add_rmsnorm.  The tuner times the form with one destination. */
typedef struct {
    const void* x;     /* device, [ring_sets][n_tokens, hidden] */
    const void* r;     /* device */
    const void* w;     /* device, [hidden] */
    void* y;           /* device; must not alias x here (launches repeat) */
    void* r_out;       /* device; must not alias r here */
    const void* y_ref; /* device, oracle y for rows [0, n_ref_tokens) of set 0 */
    const void* r_ref; /* device, oracle r' for the same rows */
    int64_t n_ref_tokens;     /* rows covered by the references, 1..n_tokens */
    int64_t ring_stride_bytes;/* distance between consecutive sets of x, r, y, r_out (0 when ring_sets == 1) */
    int32_t ring_sets;        /* >= 1; timed launches rotate over the sets (cold-L2 timing of small shapes) */
    float eps;
    void* stream;
    const void* aux;   /* device; merge_attn_states: s_b.  NULL otherwise */
    void* aux_out;     /* device; fp8-output norm: the per-token scales.  NULL otherwise */
    const void* aux_ref; /* device; reference for aux_out */
} rt_workspace;

typedef enum { RT_PHASE_SEED = 0, RT_PHASE_GRID = 1, RT_PHASE_CLIMB = 2, RT_PHASE_TOPK = 3,
               RT_PHASE_SWEEP = 4 } rt_phase;

/* One line of the search log: every evaluated theta, its gate result and its time. */
typedef struct {
    rt_params params;
    int32_t phase;      /* rt_phase */
    int32_t eval_index; /* 0-based order of evaluation */
    int32_t status;     /* RT_OK, RT_ERR_MISMATCH, RT_ERR_CUDA, ... for this candidate */
    int32_t y_max_ulp;  /* 16-bit dtypes: worst distance of y from the reference in ulps */
    int64_t y_bad;      /* elements of y beyond tolerance */
    int64_t r_bad;      /* elements of r_out whose bits differ from the reference */
    float y_max_rel;    /* fp32: worst relative error of y */
    float us;           /* score: median over blocks of (block time / iters), microseconds */
    float us_min_block; /* fastest block */
    float us_mean;      /* mean over all blocks */
    int32_t occupancy_blocks_per_sm;
    int32_t regs_per_thread;
} rt_eval_record;

typedef struct {
    rt_params best;
    float best_us;
    int32_t evals_used;
    int32_t n_candidates; /* size of the feasible set searched */
    int32_t n_log;        /* records written to the caller's log (<= log_cap) */
    int32_t n_failed_gate;
} rt_result;

typedef enum {
    RT_OK = 0,
    RT_ERR_NULL = 1,           /* a required pointer is NULL */
    RT_ERR_DTYPE = 2,
    RT_ERR_SHAPE = 3,          /* n_tokens < 0, hidden <= 0, hidden too large */
    RT_ERR_ALIGN = 4,          /* a pointer or the row length is not a multiple of vec_bytes (or of 16 for TMA);
                                  RT_STAGE_REG_REALIGN constrains the pointers only */
    RT_ERR_INFEASIBLE = 5,     /* theta violates a hard limit; nothing was launched.  Also the answer for rows longer
                                  than any theta can serve: a row is reduced in one pass by one CTA or one cluster,
                                  so it must fit on chip.  The longest rows are served by RT_STAGE_SMEM_LDG, which
                                  keeps the row as fp32 in up to 227 KB of shared memory: 57 856 elements in one CTA
                                  and 462 336 split over a cluster of 8, for every dtype (the register stages hold
                                  at most 128 elements per thread within 64 K registers per CTA, i.e. 32 768).
                                  There is no multi-pass fall-back for longer rows (hidden sizes of language models
                                  are an order of magnitude and more below the limit) */
    RT_ERR_CUDA = 6,           /* a CUDA runtime call failed; see rt_last_error() */
    RT_ERR_MISMATCH = 7,       /* correctness gate failed (search: for every candidate) */
    RT_ERR_BUDGET = 8,         /* the budget allows no evaluation */
    RT_ERR_DEVICE_TIMEOUT = 9, /* a bounded device-side wait expired (read through rt_device_status) */
    RT_ERR_CAPACITY = 10,      /* a caller-provided array or workspace is too small */
    RT_ERR_NO_DEVICE = 11      /* no CUDA device is available */
} rt_status;

/* ---- 1. the template kernel ------------------------------------------------- */

/*
 * Instantiate(S~, theta) and launch it (Algorithm 1, Level 2; operator as defined at
 * the top of this file).  Asynchronous on `stream`.
 *   p        host; checked against the hard feasibility rules first - an infeasible
 *            theta returns RT_ERR_INFEASIBLE / RT_ERR_ALIGN and launches nothing.
 *   x, r, w  device, read only.   y, r_out  device, written.
 *   Allowed aliasing: y == x and/or r_out == r (in-place use); any other overlap
 *   is undefined.  n_tokens == 0 is a successful no-op.
 *   Allocates nothing and never synchronises.
 */
int rmsnorm_template_launch(const rt_params* p, const void* x, const void* r, const void* w, void* y,
                            void* r_out, int64_t n_tokens, int64_t hidden, float eps, int dtype,
                            void* stream);

/*
 * The same operator on HOST buffers: copies x, r, w to the device, launches theta, copies y and
 * r_out back, in row chunks so that the two copy directions and the kernel overlap.  `workspace`
 * is device memory of at least rmsnorm_host_workspace_bytes(...) bytes, owned by the caller; host
 * buffers should be page-locked for the copies to be asynchronous.  Synchronises `stream` before
 * returning.  (End-to-end entry point; no counterpart in the paper, which times kernels only.)
 */
int rmsnorm_template_run_host(const rt_params* p, const void* x_host, const void* r_host,
                              const void* w_host, void* y_host, void* r_out_host, int64_t n_tokens,
                              int64_t hidden, float eps, int dtype, void* workspace,
                              int64_t workspace_bytes, int64_t chunk_tokens, void* stream);
/* chunk_tokens <= 0 picks rows worth about 16 MB per tensor, the fastest chunk measured over PCIe Gen5 x16. */
int64_t rmsnorm_host_workspace_bytes(int64_t n_tokens, int64_t hidden, int dtype, int64_t chunk_tokens);

/*
 * The gated activation silu_and_mul as an instance of its own template (second kernel of the paper's
 * "Kernels" list; axes: threads per row, rows per CTA, vec_bytes, unroll, stage = registers or TMA bulk;
 * it has no reduction: reduce must be RT_REDUCE_SHFL and cluster_size 1).
 *   x    device, [n_tokens, 2*d]: gate in the first d columns of a row, value in the last d.
 *   out  device, [n_tokens, d];  out = round_dtype(silu(gate) * value), silu(g) = g / (1 + exp(-g)),
 *        computed in fp32 (ex2.approx and rcp.approx: 2 ulp of a 16-bit type, 1e-5 relative in fp32).
 * Asynchronous on `stream`, allocates nothing; infeasible theta is refused without launching.
 */
int silu_and_mul_template_launch(const rt_params* p, const void* x, void* out, int64_t n_tokens, int64_t d,
                                 int dtype, void* stream);

/*
 * add_rmsnorm with a quantised output for a following fp8 GEMM (a variant of the norm template: stage =
 * registers or TMA bulk, 32- or 16-byte vectors, shuffle reduction; bf16 and fp16 inputs).  No counterpart kernel
 * in the paper; it is one of the "organization of shared memory and registers" variants its template axes
 * leave room for ("Tuning parameter selection and search space derivation").
 *   x, r, w   device, as for rmsnorm_template_launch.     r_out  device, the rounded residual (bit-exact contract).
 *   q         device, [n_tokens, hidden] bytes: e4m3 codes (4 exponent bits, bias 7, 3 significand bits, no
 *             infinities, largest finite value 448) of y / scale, round to nearest even, saturating.  Aligned to
 *             vec_bytes / 2 bytes (8 or 16; RT_ERR_ALIGN otherwise).
 *   scale     device, [n_tokens] binary32: max(max_j |y_j|, 1e-12) / 448 with y the un-rounded norm output.
 * Asynchronous on `stream`, allocates nothing; infeasible theta is refused without launching.
 */
int rmsnorm_fp8_template_launch(const rt_params* p, const void* x, const void* r, const void* w, void* q,
                                float* scale, void* r_out, int64_t n_tokens, int64_t hidden, float eps, int dtype,
                                void* stream);

/*
 * The tensor-parallel form of add_rmsnorm: the all-reduce that precedes the operator in tensor-parallel
 * serving is folded into the kernel (a variant of the norm template: register stage, 32- or 16-byte vectors, shuffle
 * reduction; axes threads per row, rows per CTA, unroll).  No counterpart in the paper, whose experiments run
 * on one GPU; the operator is its `fused_add_rmsnorm` ("Kernels") with x = sum over ranks of x^(k).
 *
 * One launch computes rows [row_begin, row_begin + row_count) of the tensors:
 *     a = fp32(x^(0));  a = a + fp32(x^(k)) for k = 1 .. n_parts-1, in this order, each a binary32 addition;
 *     s = a + fp32(r);  r_out = round_dtype(s);  y = round_dtype(s * rsqrt(mean(s^2) + eps) * w)
 * and writes those rows of y into EVERY y destination and those rows of r_out into EVERY r_out destination.
 * With rank k of an n-rank group calling it on its own block of rows, with all ranks' partials as x_parts and
 * all ranks' y tensors as y destinations, every rank ends with the complete y (reduce-scatter + operator +
 * all-gather in one kernel, the transfers being the kernel's own loads and stores over peer-mapped memory).  The
 * residual usually has one destination, the rank's own tensor: the rank's next norm needs the residual of its
 * own rows only, so each link direction carries 2 (n-1)/n tensor sizes, as much as an all-reduce of x alone.
 * With one y destination and all rows it is the one-shot form (every rank reduces everything for itself).
 *   x_parts   HOST array of n_parts (2, 4 or 8) DEVICE pointers, part k = rank k's partial x, each a full
 *             [n_rows_total, hidden] tensor addressable from the current device (its own memory or a
 *             peer-mapped allocation); read only.
 *   r, w      device (current GPU), r a full [n_rows_total, hidden] tensor, w [hidden].
 *   y_outs    HOST array of n_y_outs (1..RT_MAX_PARTS) DEVICE pointers to full [n_rows_total, hidden] tensors;
 *   r_outs    HOST array of n_r_outs (1..RT_MAX_PARTS) such pointers.  Only the launch's rows are written.  An
 *             r_out destination may be the tensor r itself (in-place residual); no destination may be a part of x.
 *   All tensor pointers must be 16-byte aligned and the row length a multiple of 16 bytes (RT_ERR_ALIGN).
 * The kernel contains no wait: the caller orders the launch after every rank's partial is complete and lets
 * no rank read the outputs before every rank's launch has finished (a barrier of the group on both sides).
 * Asynchronous on `stream`, allocates nothing; infeasible theta is refused without launching.
 */
int rmsnorm_allreduce_template_launch(const rt_params* p, const void* const* x_parts, int32_t n_parts, const void* r,
                                      const void* w, void* const* y_outs, int32_t n_y_outs, void* const* r_outs,
                                      int32_t n_r_outs, int64_t row_begin, int64_t row_count, int64_t hidden,
                                      float eps, int dtype, void* stream);

/*
 * merge_attn_states as an instance of its own template (third kernel of the paper's "Kernels" list, shapes
 * (n, h, d); axes as for silu_and_mul: no reduction, stage = registers or TMA bulk).
 *   v_a, v_b  device, [n_tokens, heads, head_dim] of `dtype`: normalised partial attention outputs.
 *   s_a, s_b  device, [n_tokens, heads] binary32: natural log of each part's softmax denominator
 *             (-inf = that part saw no keys).
 *   v_out     device, [n_tokens, heads, head_dim];  s_out  device, [n_tokens, heads] binary32.
 *   With m = max(s_a, s_b), w = exp(s - m), D = w_a + w_b:  v_out = round_dtype((w_a v_a + w_b v_b) / D),
 *   s_out = m + ln D;  both parts empty: v_out = 0, s_out = -inf.  Computed in fp32.
 * Asynchronous on `stream`, allocates nothing; infeasible theta is refused without launching.
 */
int merge_attn_states_template_launch(const rt_params* p, const void* v_a, const float* s_a, const void* v_b,
                                      const float* s_b, void* v_out, float* s_out, int64_t n_tokens,
                                      int64_t heads, int64_t head_dim, int dtype, void* stream);

/* ---- 2. the feasible region ----------------------------------------------------- */

/* r(h) of the current CUDA device.  RT_ERR_NO_DEVICE when there is none. */
int rt_query_limits(rt_limits* out);
/* Documented sm_100a (B200) limits, for host-only use (have_device = 0). */
void rt_limits_sm100_nominal(rt_limits* out);

/*
 * DeriveFeasibleSpace(S~, h, r(h)) (Algorithm 1; "Tuning parameter selection and search space
 * derivation": ranges and discrete candidate sets from the hardware limits, pruning combinations
 * that would not compile, not launch, or be obviously inefficient).
 *   s      host.   out  host array of `cap` entries (may be NULL when cap == 0).
 *   *n_out receives the size of the feasible set, which may exceed `cap`: call twice.
 * Uses the current device's limits and, for every candidate, the compiled kernel's register count,
 * spill size and occupancy.  tuner_derive_feasible_ex takes the limits and the heuristic mask
 * explicitly (limits->have_device == 0 works without a GPU).
 */
int tuner_derive_feasible(const rt_shape* s, rt_params* out, int32_t cap, int32_t* n_out);
int tuner_derive_feasible_ex(const rt_shape* s, const rt_limits* limits, int32_t heuristics,
                             rt_params* out, int32_t cap, int32_t* n_out);
/* Hard rules only, for one theta: RT_OK, RT_ERR_ALIGN or RT_ERR_INFEASIBLE (reason in rt_last_error). */
int tuner_check_params(const rt_shape* s, const rt_limits* limits, const rt_params* p);
/* The raw (unpruned) grid, for reporting how much the deriver removed. */
int tuner_raw_grid(const rt_shape* s, rt_params* out, int32_t cap, int32_t* n_out);
/*
 * How the raw grid was pruned.  counts (host, n_counts >= 11): [0..7] points removed by a hard rule,
 * by reason (0 unused, 1 arguments, 2 threads per CTA, 3 alignment, 4 registers, 5 shared memory,
 * 6 cluster, 7 grid size); [8] removed by the heuristic rules; [9] feasible; [10] raw grid size.
 */
int tuner_derive_counts(const rt_shape* s, const rt_limits* limits, int32_t heuristics, int32_t* counts,
                        int32_t n_counts);

/* ---- 3. search -------------------------------------------------------------------- */

/*
 * Search(S~, x, Theta_feasible) for one input shape (Algorithm 1): seeds first, then a coarse
 * grid over the feasible set, then best-first hill-climbing over one-step neighbours on
 * measured time (around the fastest point, then once around the fastest point of every other stage
 * that is within 3 % of it, then around the three fastest and, while budget remains, up to the
 * twelve fastest), then a re-test of the top_k finalists ("Tuning agent": Top-K re-testing): they are
 * re-timed side by side as tuner_retest_interleaved does, each counts as one evaluation, the winner is the
 * fastest finalist that passes again (re-test times within 0.5 % of the fastest are a tie, which goes to the finalist
 * that was faster when the search first timed it), and a finalist that fails its re-test is replaced by the next runner-up
 * while budget remains.
 * Every candidate passes the correctness gate (r_out bit-exact, y within 2 ulp for 16-bit types or
 * 1e-5 relative for fp32, against the uploaded references) before it is timed; candidates that
 * fail the gate or the launch are logged and skipped.
 *   log      host array of log_cap records (may be NULL).   Synchronises the stream repeatedly.
 *   Allocates a few bytes of device memory on first use (freed by rt_shutdown).
 * RT_ERR_MISMATCH when no candidate passed the gate; RT_ERR_BUDGET when max_evals < 1.
 */
int tuner_search(const rt_shape* s, const rt_budget* b, const rt_workspace* ws, rt_result* out,
                 rt_eval_record* log, int32_t log_cap);

/*
 * The same search over a caller-supplied cost function instead of the device (host only; used to
 * test the search logic and budget accounting).  `evaluate` returns the time of theta in
 * microseconds, or a negative value / NaN for a candidate that fails its gate.
 */
typedef double (*rt_evaluate_fn)(const rt_params* p, void* user);
int tuner_search_with(const rt_shape* s, const rt_limits* limits, const rt_budget* b,
                      rt_evaluate_fn evaluate, void* user, rt_result* out, rt_eval_record* log,
                      int32_t log_cap);

/* Gate + timing of one theta with the protocol of `b` (warmup, iters, repeats, use_graph). */
int tuner_evaluate(const rt_shape* s, const rt_params* p, const rt_budget* b, const rt_workspace* ws,
                   rt_eval_record* out);

/* One timed block of tuner_retest_interleaved. */
typedef struct {
    int32_t theta_index; /* index into the caller's theta array */
    int32_t round;       /* 0-based round the block belongs to */
    float us;            /* block time / iters, microseconds */
    int32_t reserved;    /* 0 */
    double t_begin_s;    /* host CLOCK_MONOTONIC seconds just before the block's first timed launch ... */
    double t_end_s;      /* ... and just after its last one completed: for matching clock samples to blocks */
} rt_block_record;

/*
 * Top-K re-test as a measurement of its own ("Tuning agent": Top-K re-testing before the convergence decision;
 * protocol of "Performance Measurement" per block): several thetas re-timed side by side.  Every theta passes the
 * gate once; then `rounds` rounds follow, and in each round every theta runs one block - b->warmup untimed launches,
 * then b->iters launches between two events (one CUDA graph when b->use_graph) - before any theta runs its next
 * block; the order rotates by one from round to round.  A clock or power change during the measurement therefore
 * meets every theta alike, which back-to-back evaluations of one theta after the other do not give.
 *   thetas  host, n_thetas entries.      out  host, n_thetas records: status and gate statistics of theta i,
 *           us = median over its blocks, us_min_block, us_mean.  A theta that is refused or fails the gate has
 *           its status set and takes no further part.
 *   blocks  host, rounds * n_thetas records, or NULL: every block in the order it ran (fewer when thetas drop out;
 *           *n_blocks, may be NULL, receives the count).
 * tuner_search runs its own Top-K confirmation through the same routine (rounds = b->repeats).  Synchronises the
 * stream repeatedly.
 */
int tuner_retest_interleaved(const rt_shape* s, const rt_params* thetas, int32_t n_thetas, const rt_budget* b,
                             const rt_workspace* ws, int32_t rounds, rt_eval_record* out, rt_block_record* blocks,
                             int32_t* n_blocks);

/*
 * Time of an empty kernel under the same protocol (warmup, iters, repeats, use_graph of `b`), in
 * microseconds per launch: the floor below which no candidate of a latency-bound shape can score.
 * Synchronises `stream`.  (Measurement aid for "Performance Measurement"; the paper has no counterpart.)
 */
int tuner_launch_floor(const rt_budget* b, void* stream, float* us);

/*
 * rmsnorm_template_launch through an instrumented instance of the same template, for the latency-bound shapes
 * (measurement aid; "Performance Measurement" in the paper times whole kernels only).  The first thread of every CTA
 * records, into RT_TRACE_WORDS 64-bit words at trace[cta * RT_TRACE_WORDS]:
 *   [0] the global nanosecond timer at kernel entry      [6] the same timer just before the CTA exits
 *   [1] SM cycle counter at entry                        [2] ... once the previous kernel of the stream has completed
 *   [3] ... once the thread's share of x and r has arrived and been summed
 *   [4] ... once the row's sum of squares is reduced     [5] ... once the thread's last store has been issued
 *   [7] the SM the CTA ran on.
 * Cycle counts of one CTA are comparable with each other (one SM); the nanosecond timer is comparable across CTAs and
 * launches but ticks coarsely.  Instrumented instances exist for bf16 and fp32 with vec_bytes = 16 and unroll 1: the
 * register stage with at most two vectors per thread (all three reductions for bf16 with one vector per thread) and,
 * for bf16, the TMA stage; any other theta returns RT_ERR_INFEASIBLE.  trace: device, trace_words >= the value
 * rmsnorm_trace_words returns for this theta and shape (RT_ERR_CAPACITY otherwise; -1 from rmsnorm_trace_words when
 * theta is infeasible).  Outputs are the operator's, as from rmsnorm_template_launch.  Asynchronous, allocates nothing.
 */
#define RT_TRACE_WORDS 8
int rmsnorm_template_launch_traced(const rt_params* p, const void* x, const void* r, const void* w, void* y, void* r_out,
                                   int64_t n_tokens, int64_t hidden, float eps, int dtype, uint64_t* trace,
                                   int64_t trace_words, void* stream);
int64_t rmsnorm_trace_words(const rt_params* p, int64_t n_tokens, int64_t hidden, int dtype);

/* ---- 4. general configuration and specialised table -------------------------------------- */

/* One row of D_spec: a shape and the best theta found for it. */
typedef struct {
    rt_shape shape;
    rt_params best;
    float best_us;
    int32_t reserved;
} rt_spec_entry;

typedef enum { RT_FROM_TABLE_EXACT = 0, RT_FROM_TABLE_NEAREST = 1, RT_FROM_GENERAL = 2,
               RT_FROM_FEASIBLE_SET = 3 } rt_theta_source;

/*
 * SelectGeneral (Algorithm 1; "Performance Measurement": the general configuration is the one with the
 * best average performance across shapes).  Host only.
 *   times_us  host, [n_candidates][n_shapes], the measured time of candidate c on shape x; a value <= 0,
 *             NaN or inf marks "could not run / failed its gate on that shape".
 * With T*(x) the best time on shape x over all candidates, the score of a candidate is the geometric mean
 * over shapes of T*(x) / T(theta, x) (the paper's geometric-mean speedup with the per-shape optimum as the
 * reference; 1.0 = best everywhere).  A candidate that cannot run on some shape scores 0 and is not
 * eligible.  *best_index receives the eligible candidate with the highest score (first on ties);
 * scores (may be NULL) receives every candidate's score.  RT_ERR_INFEASIBLE when none is eligible.
 */
int tuner_select_general(const float* times_us, int32_t n_candidates, int32_t n_shapes, int32_t* best_index,
                         float* best_score, float* scores);

/*
 * BuildSpecialized's table put to use: theta for a query shape.  Host only (limits == NULL asks the
 * current device).  Order of preference: the table entry of the same element size nearest to the query (distance
 * = 4 x octaves of hidden size + octaves of token count + 2 x octaves of head size where the kernel has
 * heads, + 0.25 for a bf16 entry serving an fp16 query or the reverse; distance 0 is an exact hit) whose theta passes the
 * hard feasibility rules for the query; else `general` (may be NULL) if feasible; else the first point
 * of the derived feasible set.  *source (may be NULL) receives an rt_theta_source.
 */
int tuner_table_lookup(const rt_spec_entry* table, int32_t n_entries, const rt_params* general,
                       const rt_shape* query, const rt_limits* limits, rt_params* out, int32_t* source);

/*
 * rmsnorm_template_launch with theta taken from tuner_table_lookup for this call's shape and pointer
 * alignment.  `used` (may be NULL) receives the theta launched.  Asynchronous, allocates nothing.
 * Each thread remembers its last lookup (table address, entry count, shape), so a loop over one shape pays for
 * the lookup once: do not edit a table in place while it is in use - build a new array instead.
 */
int rmsnorm_launch_auto(const rt_spec_entry* table, int32_t n_entries, const rt_params* general,
                        const void* x, const void* r, const void* w, void* y, void* r_out, int64_t n_tokens,
                        int64_t hidden, float eps, int dtype, void* stream, rt_params* used);

typedef enum { RT_CMP_BITS = 0, RT_CMP_ULP16 = 1, RT_CMP_REL32 = 2 } rt_compare_mode;
/*
 * d(.,.) for e4m3 codes: distance in code steps on the format's value lattice (+0 == -0, NaN matches NaN).
 * got, ref: device, n bytes.  *max_steps, *n_bad (elements beyond tol_steps): host.  Synchronises `stream`.
 */
int tuner_compare_e4m3(const void* got, const void* ref, int64_t n, int32_t tol_steps, int32_t* max_steps,
                       int64_t* n_bad, void* stream);
/*
 * d(.,.) for outputs that may cancel (merge_attn_states): an element passes when it is within `tol` of the
 * reference - units in the last place for the 16-bit types, relative for binary32 - OR within `tol_abs`
 * absolutely.  *max_abs receives the largest absolute difference, *n_bad the failing elements.
 * got, ref: device; max_abs, n_bad: host.  Synchronises `stream`.
 */
int tuner_compare_mixed(const void* got, const void* ref, int64_t n, int dtype, double tol, double tol_abs,
                        double* max_abs, int64_t* n_bad, void* stream);
/*
 * The distance d(.,.) of the correctness criterion, computed on the device.
 *   got, ref  device, n elements of `dtype`.
 *   RT_CMP_BITS : *n_bad = elements whose bit patterns differ; *max_err = 1 if any.
 *   RT_CMP_ULP16: distance in units of the last place on the 16-bit type's value lattice
 *                 (+0 == -0, NaN matches NaN); *n_bad = elements beyond `tol`.
 *   RT_CMP_REL32: |got-ref| <= tol*|ref| + 1e-30 for fp32; *max_err = worst |got-ref|/|ref|.
 *   max_err, n_bad: host.  Synchronises `stream`.  The comparison entry points (this one, _mixed, _e4m3) and
 *   the tuner's evaluations share one accumulator block per device and are serialised by a lock.
 */
int tuner_compare(const void* got, const void* ref, int64_t n, int dtype, int mode, double tol,
                  double* max_err, int64_t* n_bad, void* stream);

/*
 * tuner_compare without any allocation.  (No counterpart in the paper: it exists for callers that
 * cannot allocate device memory.)
 *
 * Some callers must not reach cudaMalloc at all: a serving process that has handed the whole device
 * to its own memory pool (a raw allocation there fails, or takes memory the pool counts on), and code
 * on a latency path where the device-wide synchronisation that cudaMalloc and cudaFree imply is not
 * acceptable.  tuner_compare allocates its accumulator (device and page-locked host memory) on first
 * use; this entry point calls no cudaMalloc, cudaMallocHost, cudaFree or any other allocating routine,
 * now or later.  Arguments, modes, results and errors are those of tuner_compare.
 *
 * Its accumulator lives in a fixed 256-byte array inside the library's device image: every GPU that
 * loads the library holds those 256 bytes until the process exits.  The accumulator does not grow with
 * n; n is limited to 2^40 elements (RT_ERR_CAPACITY beyond that, nothing is launched).
 *
 * The first call on each device looks up the array's device address (with that device current); make
 * that first call before starting any stream capture.  All calls on a device share the one array: it is
 * cleared at the start of every call, so calls in a row are independent, but two calls whose work
 * overlaps on the GPU (different streams, different threads) race on it and return garbage - serialise
 * them.  Synchronises `stream`.
 */
int tuner_compare_static(const void* got, const void* ref, int64_t n, int dtype, int mode, double tol,
                         double* max_err, int64_t* n_bad, void* stream);

/* ---- housekeeping ------------------------------------------------------------------- */

const char* rt_status_string(int status);
const char* rt_last_error(void);
/* Reads and clears the device status word (0, or RT_ERR_DEVICE_TIMEOUT).  Synchronises the device. */
int rt_device_status(void);
/* Number of compiled instances of the template, and the i-th one's coordinates (host query). */
int32_t rt_num_kernel_instances(void);
int rt_kernel_instance(int32_t i, int32_t* dtype, int32_t* vec_bytes, int32_t* stage, int32_t* reduce,
                       int32_t* unroll, int32_t* reg_vectors);
/* The rt_op the i-th instance belongs to (-1 when i is out of range). */
int32_t rt_kernel_instance_op(int32_t i);
/* Partial inputs the i-th instance sums per element (all-reduce-fused norm; 0 for the others, -1 out of range). */
int32_t rt_kernel_instance_parts(int32_t i);
/*
 * Process-wide launch options.  RT_OPTION_PROGRAMMATIC_LAUNCH (0 or 1, default 1): launch every kernel of the
 * library with the programmatic-stream-serialization attribute, so that a launch's CTAs may be scheduled, and
 * run their prologue, while the previous kernel of the stream is still finishing; each kernel waits
 * (griddepcontrol.wait) for that kernel to complete, and for its writes to be visible, before it touches memory,
 * so results do not depend on the option.  Measured on B200: 10-13% on the latency-bound shapes inside a CUDA
 * graph, 40% on them in a plain stream of launches, 1-3.5% on the bandwidth-bound shapes.  Set it to 0 to launch
 * with full stream serialization.
 * rt_set_option returns RT_ERR_SHAPE for an unknown option or value; rt_get_option returns -1 for an unknown option.
 *
 * RT_OPTION_TMA_WAIT_POLL_LIMIT (1 .. 2^24, default 2^24): how many times a thread of add_rmsnorm's TMA stages polls
 * its row's mbarrier before it gives up, writes RT_ERR_DEVICE_TIMEOUT into the device status word, waits once more
 * with the same limit and then carries on to every barrier of the CTA (the launch completes; its outputs are not
 * valid).  The default is about a second of polling; a copy that has not landed by then never will.
 * RT_OPTION_DEBUG_DROP_TMA_COPIES (0 or 1, default 0): diagnostic switch for exercising that path without a
 * fault - the TMA stages of add_rmsnorm initialise their mbarriers but post no copy, so every wait runs out at the
 * poll limit and the launch reports RT_ERR_DEVICE_TIMEOUT.  Nothing out of bounds is read or written.  Lower the
 * poll limit to a few thousand first, or every row waits the full default.
 */
enum { RT_OPTION_PROGRAMMATIC_LAUNCH = 0, RT_OPTION_TMA_WAIT_POLL_LIMIT = 1, RT_OPTION_DEBUG_DROP_TMA_COPIES = 2 };
int rt_set_option(int32_t option, int32_t value);
int32_t rt_get_option(int32_t option);
/* Kernel launches issued by this library in this process since load (all entry points). */
int64_t rt_launch_count(void);
/* Frees what the library allocated on the device.  Safe to call more than once. */
void rt_shutdown(void);

#ifdef __cplusplus
}
#endif
#endif /* RMSNORM_TUNER_H_ */
