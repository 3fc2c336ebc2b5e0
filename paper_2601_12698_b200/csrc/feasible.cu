// DeriveFeasibleSpace(S~, h, r(h)): the raw parameter grid, the hard rules (make_plan) and the
// switchable "obvious inefficiency" rules, after the paper's Section "Tuning parameter selection and
// search space derivation".
#include <string.h>

#include "tuner_internal.h"

namespace rt {

namespace {

const int kTprLevels[] = {32, 64, 128, 256, 512, 1024};
const int kRpcLevels[] = {1, 2, 4, 8};
const int kUnrollLevels[] = {1, 2, 4};
struct Mode {
    int reduce, cluster;
};
const Mode kReduceModes[] = {{RT_REDUCE_SHFL, 1}, {RT_REDUCE_SMEM, 1}, {RT_REDUCE_CLUSTER, 2},
                             {RT_REDUCE_CLUSTER, 4}, {RT_REDUCE_CLUSTER, 8}};

int next_pow2(int v)
{
    int p = 1;
    while (p < v) p <<= 1;
    return p;
}

// Vector widths offered for a shape: 32, 16 and 8 bytes (the tuned axis); when the row length or a base
// pointer allows neither, the widest narrower width that fits (a fall-back, not a tuned axis).
std::vector<int> vec_levels(const rt_shape& s)
{
    const int eb = elem_bytes_of(s.dtype);
    const int64_t row_bytes = s.hidden * eb;
    const int64_t head_bytes = s.op == RT_OP_MERGE_ATTN_STATES && s.head_dim > 0 ? (int64_t)s.head_dim * eb : row_bytes;
    auto fits = [&](int vb) { return vb >= eb && row_bytes % vb == 0 && head_bytes % vb == 0 && s.min_ptr_align >= vb; };
    if (fits(32) || fits(16) || fits(8)) {
        return {32, 16, 8};  // 32: the 256-bit global accesses of sm_100
    }
    if (fits(4)) return {4};
    if (fits(2)) return {2};
    return {16, 8};  // nothing fits: the hard rules reject every point and say why
}

}  // namespace

uint64_t pack_params(const rt_params& p)
{
    return ((uint64_t)(uint16_t)p.threads_per_row) | ((uint64_t)(uint8_t)p.rows_per_cta << 16) |
           ((uint64_t)(uint8_t)p.vec_bytes << 24) | ((uint64_t)(uint8_t)p.unroll << 32) |
           ((uint64_t)(uint8_t)p.stage << 40) | ((uint64_t)(uint8_t)p.reduce << 44) |
           ((uint64_t)(uint8_t)p.cluster_size << 48);
}

std::vector<rt_params> raw_grid(const rt_shape& s)
{
    std::vector<rt_params> out;
    const std::vector<int> vecs = vec_levels(s);
    // silu_and_mul and merge_attn_states have no reduction and no ld.global -> shared stage: their grid is
    // the remaining axes
    const bool is_silu = s.op == RT_OP_SILU_AND_MUL || s.op == RT_OP_MERGE_ATTN_STATES;  // no reduction axis
    const int kStages[] = {RT_STAGE_REG, RT_STAGE_SMEM_LDG, RT_STAGE_SMEM_TMA, RT_STAGE_TMA_PIPELINE};
    for (int stage : kStages)
        for (const Mode& m : kReduceModes)
            for (int vb : vecs) {
                // the persistent pipeline: add_rmsnorm only, a row stays inside one CTA
                if (stage == RT_STAGE_TMA_PIPELINE && (s.op != RT_OP_ADD_RMSNORM || m.cluster != 1)) continue;
                if (is_silu && (stage == RT_STAGE_SMEM_LDG || m.reduce != RT_REDUCE_SHFL)) continue;
                // the fp8-output norm: 32- or 16-byte vectors, shuffle reduction, register or TMA stage
                if (s.op == RT_OP_ADD_RMSNORM_FP8 && (stage == RT_STAGE_SMEM_LDG || m.reduce != RT_REDUCE_SHFL || vb < 16))
                    continue;
                // the all-reduce-fused norm: 32- or 16-byte vectors, shuffle reduction, register stage
                if (s.op == RT_OP_ADD_RMSNORM_ALLREDUCE && (stage != RT_STAGE_REG || m.reduce != RT_REDUCE_SHFL || vb < 16))
                    continue;
                for (int tpr : kTprLevels)
                    for (int rpc : kRpcLevels)
                        for (int u : kUnrollLevels) {
                            rt_params p;
                            p.threads_per_row = tpr;
                            p.rows_per_cta = rpc;
                            p.vec_bytes = vb;
                            p.unroll = u;
                            p.stage = stage;
                            p.reduce = m.reduce;
                            p.cluster_size = m.cluster;
                            out.push_back(p);
                        }
            }
    // Rows whose byte length is not a multiple of 32 (or of 16) also get the ragged-row register stage with 32-byte
    // (and 16-byte) chunks, which keeps wide accesses on such rows; on rows that the chunk width divides it would only
    // repeat the register stage with extra bookkeeping.
    for (int chunk : {32, 16}) {
        if (s.op != RT_OP_ADD_RMSNORM || (s.hidden * elem_bytes_of(s.dtype)) % chunk == 0) continue;
        for (int tpr : kTprLevels)
            for (int rpc : kRpcLevels)
                for (int u : kUnrollLevels) {
                    rt_params p;
                    p.threads_per_row = tpr;
                    p.rows_per_cta = rpc;
                    p.vec_bytes = chunk;
                    p.unroll = u;
                    p.stage = RT_STAGE_REG_REALIGN;
                    p.reduce = RT_REDUCE_SHFL;
                    p.cluster_size = 1;
                    out.push_back(p);
                }
    }
    return out;
}

// Bytes of input an SM has in flight at once under theta: resident CTAs x what one CTA asks for before it
// consumes anything (a whole row slice per input for the bulk-copy stages, one batch of `unroll` vectors per
// thread and input otherwise).  0 when the rule below does not apply: fewer than two waves of CTAs (the batch, not
// theta, bounds what is in flight), the fall-back vector widths (nothing wider exists for the shape), and
// merge_attn_states (rows of one head: its CTAs are bound by their count, not by what each one loads).
static int64_t load_bytes_in_flight_per_sm(const rt_shape& s, const rt_limits& L, const rt_params& p, const Plan& plan,
                                           int occupancy)
{
    if (s.op == RT_OP_MERGE_ATTN_STATES || p.vec_bytes < 8 || occupancy < 1) return 0;
    if ((int64_t)plan.grid_x < 2 * (int64_t)L.sm_count * occupancy) return 0;
    const int64_t slice_bytes = (int64_t)plan.slice_nvec * p.vec_bytes * p.rows_per_cta;
    const int inputs = s.op == RT_OP_ADD_RMSNORM_ALLREDUCE ? s.n_parts + 1 : 2;  // x and r; gate and up; the parts and r
    int64_t per_cta = slice_bytes;
    if (p.stage == RT_STAGE_TMA_PIPELINE)
        per_cta = slice_bytes * p.unroll;
    else if (p.stage != RT_STAGE_SMEM_TMA)
        per_cta = std::min<int64_t>(slice_bytes, (int64_t)p.threads_per_row * p.rows_per_cta * p.vec_bytes * p.unroll);
    return per_cta * inputs * occupancy;
}

// Little's law on the loads: DRAM read bandwidth x latency under load is what the whole GPU must have in flight
// (about 3.3 TB/s of reads x 0.7-1 us = 2.3-3.3 MB on B200, 16-22 KB per SM) before bandwidth, not latency, bounds the
// kernel.  Measured on 59 exhaustive sweeps of bandwidth-bound shapes (bf16, fp16, fp32; 1024 to 32768 rows of 4096 to
// 14336 elements): of the 7579 points below 32 KB per SM none came within 21 % of its shape's optimum.
constexpr int64_t kMinLoadBytesInFlightPerSm = 32 * 1024;

// The heuristic rules.  Returns the RT_PRUNE_* bit of the first rule that removes theta, or 0.
static int heuristic_reject(const rt_shape& s, const rt_limits& L, const rt_params& p, const Plan& plan, int mask)
{
    // Threads that never own a vector: pruned once half the row's threads or more are idle, i.e. the next smaller
    // level already gives every vector a thread of its own.  The level in between stays: 320 vectors on 512 threads
    // (one vector per thread, 192 threads idle) measured 5 % faster than the same row on 256 threads on bf16/fp16
    // 32 x 5120, and level with it on fp16 8192 x 7168.  A row narrower than one warp keeps the smallest row width:
    // something must remain feasible.
    if ((mask & RT_PRUNE_IDLE_THREADS) && p.threads_per_row > std::max(next_pow2(plan.slice_nvec), L.warp_size))
        return RT_PRUNE_IDLE_THREADS;
    if ((mask & RT_PRUNE_PIPELINE_STAGE) && p.stage == RT_STAGE_TMA_PIPELINE) return RT_PRUNE_PIPELINE_STAGE;
    if (mask & RT_PRUNE_DUPLICATES) {
        if (p.stage == RT_STAGE_TMA_PIPELINE) {
            // a ring deeper than the row blocks a CTA walks over never fills
            if (p.unroll > next_pow2(plan.blocks_per_cta)) return RT_PRUNE_DUPLICATES;
        } else if (p.unroll > next_pow2(plan.vec_per_thread)) {
            return RT_PRUNE_DUPLICATES;  // a batch deeper than the vectors a thread owns only adds predicated-off slots
        }
    }
    if ((mask & RT_PRUNE_CLUSTER_WAVES) && p.cluster_size > 1) {
        // Splitting rows is for shapes with too few rows to occupy the SMs: allow a split into C only
        // while the next smaller split still leaves SMs without a CTA.
        const int64_t row_ctas = (s.n_tokens + p.rows_per_cta - 1) / p.rows_per_cta;
        if (row_ctas * (p.cluster_size / 2) >= L.sm_count) return RT_PRUNE_CLUSTER_WAVES;
    }
    if ((mask & RT_PRUNE_IDLE_ROWS) && s.n_tokens > 0 && p.rows_per_cta > s.n_tokens) return RT_PRUNE_IDLE_ROWS;
    return 0;
}

int derive_feasible(const rt_shape& s, const rt_limits& L, int heuristics, std::vector<rt_params>* out, int32_t* counts)
{
    int32_t local[kRejectReasons + 3];
    memset(local, 0, sizeof(local));
    if (s.dtype < 0 || s.dtype > 2) {
        set_error("dtype %d is not one of bf16(0), fp16(1), fp32(2)", s.dtype);
        return RT_ERR_DTYPE;
    }
    if (s.n_tokens < 0 || s.hidden <= 0 || s.hidden * elem_bytes_of(s.dtype) >= (int64_t)1 << 31) {
        set_error("shape n_tokens=%lld hidden=%lld is out of range", (long long)s.n_tokens, (long long)s.hidden);
        return RT_ERR_SHAPE;
    }
    const std::vector<rt_params> raw = raw_grid(s);
    local[kRejectReasons + 2] = (int32_t)raw.size();
    std::vector<rt_params> kept;
    std::vector<int64_t> in_flight;  // per kept theta; 0: the bytes-in-flight rule does not apply to it
    int64_t most_in_flight = 0;
    for (const rt_params& p : raw) {
        Plan plan;
        const int st = make_plan(&s, &p, &L, &plan);
        if (st == RT_ERR_CUDA || st == RT_ERR_NO_DEVICE) return st;
        if (st != RT_OK) {
            local[plan.reject_reason < kRejectReasons ? plan.reject_reason : kRejectArgs]++;
            continue;
        }
        const int occupancy = plan_occupancy(plan, &L, nullptr);
        if (occupancy < 1) {
            local[plan.dyn_smem > 0 ? kRejectSmem : kRejectRegisters]++;
            continue;
        }
        if (heuristic_reject(s, L, p, plan, heuristics)) {
            local[kRejectReasons]++;
            continue;
        }
        kept.push_back(p);
        in_flight.push_back(load_bytes_in_flight_per_sm(s, L, p, plan, occupancy));
        most_in_flight = std::max(most_in_flight, in_flight.back());
    }
    // RT_PRUNE_BYTES_IN_FLIGHT: a theta that keeps too few bytes of loads in flight to cover DRAM latency, on a
    // shape where some other theta does (narrow rows may allow none: then the rule is void and all stay)
    const bool rule_applies = (heuristics & RT_PRUNE_BYTES_IN_FLIGHT) && most_in_flight >= kMinLoadBytesInFlightPerSm;
    for (size_t i = 0; i < kept.size(); ++i) {
        if (rule_applies && in_flight[i] > 0 && in_flight[i] < kMinLoadBytesInFlightPerSm) {
            local[kRejectReasons]++;
            continue;
        }
        local[kRejectReasons + 1]++;
        if (out) out->push_back(kept[i]);
    }
    if (counts) memcpy(counts, local, sizeof(local));
    return RT_OK;
}

}  // namespace rt

extern "C" {

int tuner_derive_feasible_ex(const rt_shape* s, const rt_limits* limits, int32_t heuristics, rt_params* out,
                             int32_t cap, int32_t* n_out)
{
    if (!s || !n_out || (cap > 0 && !out)) {
        rt::set_error("tuner_derive_feasible: NULL argument");
        return RT_ERR_NULL;
    }
    rt_limits L;
    if (!limits) {
        int st = rt::current_limits(&L);
        if (st != RT_OK) return st;
        limits = &L;
    }
    std::vector<rt_params> v;
    int st = rt::derive_feasible(*s, *limits, heuristics, &v, nullptr);
    if (st != RT_OK) return st;
    *n_out = (int32_t)v.size();
    const int32_t n_copy = std::min<int32_t>(cap, (int32_t)v.size());
    for (int32_t i = 0; i < n_copy; ++i) out[i] = v[i];
    return RT_OK;
}

int tuner_derive_feasible(const rt_shape* s, rt_params* out, int32_t cap, int32_t* n_out)
{
    return tuner_derive_feasible_ex(s, nullptr, RT_PRUNE_DEFAULT, out, cap, n_out);
}

int tuner_derive_counts(const rt_shape* s, const rt_limits* limits, int32_t heuristics, int32_t* counts, int32_t n_counts)
{
    if (!s || !counts) {
        rt::set_error("tuner_derive_counts: NULL argument");
        return RT_ERR_NULL;
    }
    if (n_counts < rt::kRejectReasons + 3) {
        rt::set_error("counts needs %d entries", rt::kRejectReasons + 3);
        return RT_ERR_CAPACITY;
    }
    rt_limits L;
    if (!limits) {
        int st = rt::current_limits(&L);
        if (st != RT_OK) return st;
        limits = &L;
    }
    return rt::derive_feasible(*s, *limits, heuristics, nullptr, counts);
}

int tuner_raw_grid(const rt_shape* s, rt_params* out, int32_t cap, int32_t* n_out)
{
    if (!s || !n_out || (cap > 0 && !out)) {
        rt::set_error("tuner_raw_grid: NULL argument");
        return RT_ERR_NULL;
    }
    const std::vector<rt_params> v = rt::raw_grid(*s);
    *n_out = (int32_t)v.size();
    const int32_t n_copy = std::min<int32_t>(cap, (int32_t)v.size());
    for (int32_t i = 0; i < n_copy; ++i) out[i] = v[i];
    return RT_OK;
}

}  // extern "C"
