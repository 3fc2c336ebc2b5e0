// SelectGeneral and BuildSpecialized of Algorithm 1: the general configuration theta_gen (one theta for all
// shapes, chosen by geometric-mean speedup as in "Performance Measurement and Evaluation") and the
// specialised table D_spec (shape -> its own best theta), with a launch entry point that consults them.
#include <math.h>
#include <string.h>

#include "tuner_internal.h"

namespace rt {

// Distance between two shapes of one element size: octaves of hidden size and of token count.  Hidden size
// weighs more: it fixes vector counts, register and shared-memory footprints; the token count only
// decides how full the machine is.  bf16 and fp16 entries are neighbours of each other (the same bytes move through
// the same instances; only the conversions differ), a quarter of an octave further away than an entry of the query's own
// type: a table tuned on bf16 decode shapes then serves fp16 ones, instead of the nearest fp16 entry however far.
static double shape_distance(const rt_shape& a, const rt_shape& b)
{
    const double dh = fabs(log2((double)a.hidden) - log2((double)b.hidden));
    const double dt = fabs(log2((double)std::max<int64_t>(a.n_tokens, 1)) - log2((double)std::max<int64_t>(b.n_tokens, 1)));
    double dd = 0.0;  // merge_attn_states: the same hidden size may be cut into heads differently
    if (a.head_dim > 0 && b.head_dim > 0) dd = fabs(log2((double)a.head_dim) - log2((double)b.head_dim));
    // all-reduce-fused norm: the part count multiplies the loads in flight per thread
    if (a.n_parts > 0 && b.n_parts > 0) dd += fabs(log2((double)a.n_parts) - log2((double)b.n_parts));
    return 4.0 * dh + dt + 2.0 * dd + (a.dtype != b.dtype ? 0.25 : 0.0);
}

int table_lookup(const rt_spec_entry* table, int32_t n, const rt_params* general, const rt_shape* query,
                 const rt_limits* limits, rt_params* out, int32_t* source)
{
    int best = -1;
    double best_d = 0.0;
    for (int32_t i = 0; i < n; ++i) {
        const rt_spec_entry& e = table[i];
        if (elem_bytes_of(e.shape.dtype) != elem_bytes_of(query->dtype) || e.shape.op != query->op) continue;
        // the ragged-row stage runs on any row length, but on rows that its chunk width divides it is the register
        // stage plus bookkeeping: an entry tuned on a misaligned shape is not a neighbour of an aligned one
        if (e.best.stage == RT_STAGE_REG_REALIGN && e.best.vec_bytes > 0 &&
            (query->hidden * elem_bytes_of(query->dtype)) % e.best.vec_bytes == 0)
            continue;
        const double d = shape_distance(e.shape, *query);
        if (best >= 0 && d >= best_d) continue;
        Plan plan;
        if (make_plan(query, &e.best, limits, &plan) != RT_OK) continue;  // not launchable on this shape
        best = i;
        best_d = d;
    }
    if (best >= 0) {
        *out = table[best].best;
        if (source) *source = best_d == 0.0 ? RT_FROM_TABLE_EXACT : RT_FROM_TABLE_NEAREST;
        return RT_OK;
    }
    if (general) {
        Plan plan;
        if (make_plan(query, general, limits, &plan) == RT_OK) {
            *out = *general;
            if (source) *source = RT_FROM_GENERAL;
            return RT_OK;
        }
    }
    // Last resort: a point of the feasible set (registers, shuffle, widest vector that fits).
    std::vector<rt_params> feasible;
    int st = derive_feasible(*query, *limits, RT_PRUNE_DEFAULT, &feasible, nullptr);
    if (st != RT_OK) return st;
    if (feasible.empty()) {
        set_error("no feasible configuration for this shape");
        return RT_ERR_INFEASIBLE;
    }
    *out = feasible[0];
    // rows that are not 16-byte multiples: the ragged-row stage near 256 threads per row, one row per CTA, deepest
    // unroll is what the searches return on such shapes, and is far ahead of the narrow row vectors
    int best_rank = -1;
    for (const rt_params& p : feasible) {
        if (p.stage != RT_STAGE_REG_REALIGN) continue;
        int away = 0;
        for (int t = p.threads_per_row; t < 256; t <<= 1) ++away;
        for (int t = p.threads_per_row; t > 256; t >>= 1) ++away;
        const int rank = 100 - 10 * away - 4 * (p.rows_per_cta - 1) + p.unroll;
        if (rank > best_rank) {
            best_rank = rank;
            *out = p;
        }
    }
    if (source) *source = RT_FROM_FEASIBLE_SET;
    return RT_OK;
}

}  // namespace rt

extern "C" {

int tuner_select_general(const float* times_us, int32_t n_candidates, int32_t n_shapes, int32_t* best_index,
                         float* best_score, float* scores)
{
    if (!times_us || !best_index) {
        rt::set_error("tuner_select_general: NULL argument");
        return RT_ERR_NULL;
    }
    if (n_candidates < 1 || n_shapes < 1) {
        rt::set_error("tuner_select_general: empty table");
        return RT_ERR_SHAPE;
    }
    // T*(x): the best time on each shape over the candidates that ran there.
    std::vector<double> best_time(n_shapes, INFINITY);
    for (int32_t c = 0; c < n_candidates; ++c)
        for (int32_t x = 0; x < n_shapes; ++x) {
            const float t = times_us[(size_t)c * n_shapes + x];
            if (t > 0.f && isfinite(t)) best_time[x] = std::min(best_time[x], (double)t);
        }
    int32_t best = -1;
    double best_s = -1.0;
    for (int32_t c = 0; c < n_candidates; ++c) {
        // geometric mean over shapes of T*(x) / T(theta, x); a candidate that cannot run somewhere is out
        double log_sum = 0.0;
        bool everywhere = true;
        for (int32_t x = 0; x < n_shapes && everywhere; ++x) {
            const float t = times_us[(size_t)c * n_shapes + x];
            if (!(t > 0.f) || !isfinite(t))
                everywhere = false;
            else
                log_sum += log(best_time[x] / (double)t);
        }
        const double score = everywhere ? exp(log_sum / n_shapes) : 0.0;
        if (scores) scores[c] = (float)score;
        if (everywhere && score > best_s) {
            best_s = score;
            best = c;
        }
    }
    if (best < 0) {
        rt::set_error("no candidate ran on every shape");
        return RT_ERR_INFEASIBLE;
    }
    *best_index = best;
    if (best_score) *best_score = (float)best_s;
    return RT_OK;
}

int tuner_table_lookup(const rt_spec_entry* table, int32_t n_entries, const rt_params* general, const rt_shape* query,
                       const rt_limits* limits, rt_params* out, int32_t* source)
{
    if (!query || !out || (n_entries > 0 && !table)) {
        rt::set_error("tuner_table_lookup: NULL argument");
        return RT_ERR_NULL;
    }
    rt_limits L;
    if (!limits) {
        int st = rt::current_limits(&L);
        if (st != RT_OK) return st;
        limits = &L;
    }
    return rt::table_lookup(table, n_entries, general, query, limits, out, source);
}

int rmsnorm_launch_auto(const rt_spec_entry* table, int32_t n_entries, const rt_params* general, const void* x,
                        const void* r, const void* w, void* y, void* r_out, int64_t n_tokens, int64_t hidden, float eps,
                        int dtype, void* stream, rt_params* used)
{
    if (n_tokens > 0 && (!x || !r || !w || !y || !r_out)) {
        rt::set_error("a tensor pointer is NULL");
        return RT_ERR_NULL;
    }
    rt_shape s = {};
    s.n_tokens = n_tokens;
    s.hidden = hidden;
    s.dtype = dtype;
    s.min_ptr_align = n_tokens > 0 ? rt::min_pointer_alignment(x, r, w, y, r_out) : 256;
    s.op = RT_OP_ADD_RMSNORM;
    s.head_dim = 0;
    // Serving loops call this with the same shape over and over: remember the last answer of this thread.
    struct Memo {
        const rt_spec_entry* table;
        const rt_params* general;
        int32_t n_entries;
        rt_shape shape;
        rt_params theta;
        bool valid;
    };
    static thread_local Memo memo = {nullptr, nullptr, 0, {}, {}, false};
    rt_params theta;
    if (memo.valid && memo.table == table && memo.general == general && memo.n_entries == n_entries &&
        memcmp(&memo.shape, &s, sizeof(s)) == 0) {
        theta = memo.theta;
    } else {
        int st = tuner_table_lookup(table, n_entries, general, &s, nullptr, &theta, nullptr);
        if (st != RT_OK) return st;
        memo = Memo{table, general, n_entries, s, theta, true};
    }
    if (used) *used = theta;
    return rmsnorm_template_launch(&theta, x, r, w, y, r_out, n_tokens, hidden, eps, dtype, stream);
}

}  // extern "C"
