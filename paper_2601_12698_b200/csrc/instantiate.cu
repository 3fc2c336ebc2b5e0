// One instantiation unit of the kernel template.  Compiled once per line of instance_units.inc with
//   -DRT_UNIT_NAME=<name> -DRT_UNIT_T=<element type> -DRT_UNIT_DTYPE=<0|1|2> -DRT_UNIT_VB=<bytes>
//   -DRT_UNIT_GROUP=<0 register stage | 1 shared-memory stages | 2 narrow fall-back | 3 silu_and_mul | 4 merge_attn_states | 5 fp8-output norm | 6 all-reduce-fused norm | 7 ragged-row register stage>
//   -DRT_UNIT_REDUCE=<0|1|2>   (register-stage units only)
//
// Instance lists.  Register stage: CAP (row vectors kept per thread) in {1,2,4,8,16,32} while the row
// stays within 128 fp32 registers per thread, unroll U in {1,2,4} with U <= CAP.  Shared-memory
// stages: U in {1,2,4}, all three reductions; the persistent pipeline stage (same units): ring depth U in
// {1,2,4}, shuffle and shared-memory reductions.  Narrow fall-back (4- and 2-byte vectors, for rows whose
// byte length is not a multiple of 8): register stage, shuffle reduction, U in {1,4}.
// Ragged-row register stage (16-byte chunks, shuffle reduction): the register stage's (CAP, U) list.
// silu_and_mul (one unit per element type, every vector width): stages register and TMA bulk for 32-, 16- and
// 8-byte vectors with U in {1,2,4}; register stage with U in {1,4} for the 4- and 2-byte fall-back.
// merge_attn_states: the same instance list as silu_and_mul.
// fp8-output norm (16-bit element types, 32- and 16-byte vectors, shuffle reduction): register stage with CAP in
// {1,2,4,8,16} (while the row stays within 128 fp32 registers per thread) and U <= CAP, TMA stage with U in {1,2,4}.
// all-reduce-fused norm (32- and 16-byte vectors, register stage, shuffle reduction): 2, 4 and 8 parts, CAP in
// {1,2,4,8,16} while the row stays within 128 fp32 registers per thread, U <= CAP with at most 256 bytes of x in flight
// per thread (U * parts <= 16 with 16-byte vectors, <= 8 with 32-byte ones).
#include "add_rmsnorm_allreduce_kernel.cuh"
#include "add_rmsnorm_fp8_kernel.cuh"
#include "add_rmsnorm_kernel.cuh"
#include "merge_attn_states_kernel.cuh"
#include "silu_and_mul_kernel.cuh"
#include "tuner_internal.h"

namespace {

using T = RT_UNIT_T;
constexpr int kDtype = RT_UNIT_DTYPE;
constexpr int kVB = RT_UNIT_VB;
constexpr int kEPV = kVB / (int)sizeof(T);
constexpr int kMaxRowRegisters = 128;

template <int ST, int RD, int U, int CAP>
rt::KernelEntry entry()
{
    constexpr bool kInRegisters = ST == rt::kStageReg || ST == rt::kStageRegRealign;
    if constexpr (kInRegisters && CAP * kEPV > kMaxRowRegisters) {
        return rt::KernelEntry{RT_OP_ADD_RMSNORM, kDtype, kVB, ST, RD, U, CAP, nullptr};  // not instantiated
    } else {
        return rt::KernelEntry{RT_OP_ADD_RMSNORM, kDtype, kVB, ST, RD, U, kInRegisters ? CAP : 0,
                               (const void*)&rt::add_rmsnorm_kernel<T, kVB, ST, RD, U, CAP>};
    }
}

template <int VB, int ST, int U>
rt::KernelEntry silu_entry()
{
    if constexpr (VB < (int)sizeof(T)) {
        return rt::KernelEntry{RT_OP_SILU_AND_MUL, kDtype, VB, ST, 0, U, 0, nullptr};  // narrower than an element
    } else {
        return rt::KernelEntry{RT_OP_SILU_AND_MUL, kDtype, VB, ST, 0, U, 0,
                               (const void*)&rt::silu_and_mul_kernel<T, VB, ST, U>};
    }
}
template <int VB, int ST, int U, int CAP>
rt::KernelEntry fp8_entry()
{
    if constexpr (sizeof(T) != 2 || (ST == rt::kStageReg && CAP * (VB / 2) > kMaxRowRegisters)) {
        return rt::KernelEntry{RT_OP_ADD_RMSNORM_FP8, kDtype, VB, ST, 0, U, CAP, nullptr};
    } else {
        return rt::KernelEntry{RT_OP_ADD_RMSNORM_FP8, kDtype, VB, ST, 0, U, ST == rt::kStageReg ? CAP : 0,
                               (const void*)&rt::add_rmsnorm_fp8_kernel<T, VB, ST, U, CAP>};
    }
}
#define RT_FP8_LIST(VB)                                                                                             \
    fp8_entry<VB, 0, 1, 1>(), fp8_entry<VB, 0, 1, 2>(), fp8_entry<VB, 0, 2, 2>(), fp8_entry<VB, 0, 1, 4>(),          \
    fp8_entry<VB, 0, 2, 4>(), fp8_entry<VB, 0, 4, 4>(), fp8_entry<VB, 0, 1, 8>(), fp8_entry<VB, 0, 2, 8>(),          \
    fp8_entry<VB, 0, 4, 8>(), fp8_entry<VB, 0, 1, 16>(), fp8_entry<VB, 0, 2, 16>(), fp8_entry<VB, 0, 4, 16>(),       \
    fp8_entry<VB, 2, 1, 1>(), fp8_entry<VB, 2, 2, 1>(), fp8_entry<VB, 2, 4, 1>()

template <int VB, int NP, int U, int CAP>
rt::KernelEntry allreduce_entry()
{
    // the row within 128 fp32 registers per thread, and at most 256 bytes of x in flight per thread
    if constexpr (CAP * (VB / (int)sizeof(T)) > kMaxRowRegisters || U * NP * VB > 256) {
        return rt::KernelEntry{RT_OP_ADD_RMSNORM_ALLREDUCE, kDtype, VB, 0, 0, U, CAP, nullptr, NP};
    } else {
        return rt::KernelEntry{RT_OP_ADD_RMSNORM_ALLREDUCE, kDtype, VB, 0, 0, U, CAP,
                               (const void*)&rt::add_rmsnorm_allreduce_kernel<T, VB, NP, U, CAP>, NP};
    }
}
#define RT_ALLREDUCE_LIST(VB, NP)                                                                                      \
    allreduce_entry<VB, NP, 1, 1>(), allreduce_entry<VB, NP, 1, 2>(), allreduce_entry<VB, NP, 2, 2>(),                  \
    allreduce_entry<VB, NP, 1, 4>(), allreduce_entry<VB, NP, 2, 4>(), allreduce_entry<VB, NP, 4, 4>(),                  \
    allreduce_entry<VB, NP, 1, 8>(), allreduce_entry<VB, NP, 2, 8>(), allreduce_entry<VB, NP, 4, 8>(),                  \
    allreduce_entry<VB, NP, 1, 16>(), allreduce_entry<VB, NP, 2, 16>(), allreduce_entry<VB, NP, 4, 16>()

template <int VB, int ST, int U>
rt::KernelEntry merge_entry()
{
    if constexpr (VB < (int)sizeof(T)) {
        return rt::KernelEntry{RT_OP_MERGE_ATTN_STATES, kDtype, VB, ST, 0, U, 0, nullptr};
    } else {
        return rt::KernelEntry{RT_OP_MERGE_ATTN_STATES, kDtype, VB, ST, 0, U, 0,
                               (const void*)&rt::merge_attn_states_kernel<T, VB, ST, U>};
    }
}
#define RT_MERGE_WIDE(VB) \
    merge_entry<VB, 0, 1>(), merge_entry<VB, 0, 2>(), merge_entry<VB, 0, 4>(), merge_entry<VB, 2, 1>(), \
    merge_entry<VB, 2, 2>(), merge_entry<VB, 2, 4>()
#define RT_SILU_WIDE(VB) \
    silu_entry<VB, 0, 1>(), silu_entry<VB, 0, 2>(), silu_entry<VB, 0, 4>(), silu_entry<VB, 2, 1>(), \
    silu_entry<VB, 2, 2>(), silu_entry<VB, 2, 4>()

#define RT_REG_LIST(RD)                                                                                   \
    entry<0, RD, 1, 1>(), entry<0, RD, 1, 2>(), entry<0, RD, 2, 2>(), entry<0, RD, 1, 4>(), entry<0, RD, 2, 4>(), \
    entry<0, RD, 4, 4>(), entry<0, RD, 1, 8>(), entry<0, RD, 2, 8>(), entry<0, RD, 4, 8>(), entry<0, RD, 1, 16>(), \
    entry<0, RD, 2, 16>(), entry<0, RD, 4, 16>(), entry<0, RD, 1, 32>(), entry<0, RD, 2, 32>(), entry<0, RD, 4, 32>()
#define RT_REALIGN_LIST                                                                                   \
    entry<3, 0, 1, 1>(), entry<3, 0, 1, 2>(), entry<3, 0, 2, 2>(), entry<3, 0, 1, 4>(), entry<3, 0, 2, 4>(), \
    entry<3, 0, 4, 4>(), entry<3, 0, 1, 8>(), entry<3, 0, 2, 8>(), entry<3, 0, 4, 8>(), entry<3, 0, 1, 16>(), \
    entry<3, 0, 2, 16>(), entry<3, 0, 4, 16>(), entry<3, 0, 1, 32>(), entry<3, 0, 2, 32>(), entry<3, 0, 4, 32>()
#define RT_SMEM_LIST(ST)                                                                                   \
    entry<ST, 0, 1, 1>(), entry<ST, 0, 2, 1>(), entry<ST, 0, 4, 1>(), entry<ST, 1, 1, 1>(), entry<ST, 1, 2, 1>(), \
    entry<ST, 1, 4, 1>(), entry<ST, 2, 1, 1>(), entry<ST, 2, 2, 1>(), entry<ST, 2, 4, 1>()

// the persistent pipeline: U is the ring depth; shuffle and shared-memory reductions
#define RT_PIPELINE_LIST                                                                                      \
    entry<4, 0, 1, 1>(), entry<4, 0, 2, 1>(), entry<4, 0, 4, 1>(), entry<4, 1, 1, 1>(), entry<4, 1, 2, 1>(), \
    entry<4, 1, 4, 1>()

std::vector<rt::KernelEntry> build_entries()
{
    std::vector<rt::KernelEntry> all = {
#if RT_UNIT_GROUP == 0
        RT_REG_LIST(RT_UNIT_REDUCE)
#elif RT_UNIT_GROUP == 1
        RT_SMEM_LIST(1), RT_SMEM_LIST(2), RT_PIPELINE_LIST
#elif RT_UNIT_GROUP == 3
        RT_SILU_WIDE(32), RT_SILU_WIDE(16), RT_SILU_WIDE(8), silu_entry<4, 0, 1>(), silu_entry<4, 0, 4>(), silu_entry<2, 0, 1>(),
        silu_entry<2, 0, 4>()
#elif RT_UNIT_GROUP == 5
        RT_FP8_LIST(32), RT_FP8_LIST(16)
#elif RT_UNIT_GROUP == 6
        RT_ALLREDUCE_LIST(32, 2), RT_ALLREDUCE_LIST(32, 4), RT_ALLREDUCE_LIST(32, 8), RT_ALLREDUCE_LIST(16, 2),
        RT_ALLREDUCE_LIST(16, 4), RT_ALLREDUCE_LIST(16, 8)
#elif RT_UNIT_GROUP == 7
        RT_REALIGN_LIST
#elif RT_UNIT_GROUP == 4
        RT_MERGE_WIDE(32), RT_MERGE_WIDE(16), RT_MERGE_WIDE(8), merge_entry<4, 0, 1>(), merge_entry<4, 0, 4>(), merge_entry<2, 0, 1>(),
        merge_entry<2, 0, 4>()
#else
        entry<0, 0, 1, 1>(), entry<0, 0, 1, 2>(), entry<0, 0, 1, 4>(), entry<0, 0, 4, 4>(), entry<0, 0, 1, 8>(),
        entry<0, 0, 4, 8>(), entry<0, 0, 1, 16>(), entry<0, 0, 4, 16>(), entry<0, 0, 1, 32>(), entry<0, 0, 4, 32>()
#endif
    };
    std::vector<rt::KernelEntry> kept;
    for (const rt::KernelEntry& e : all)
        if (e.fn) kept.push_back(e);
    return kept;
}

}  // namespace

#define RT_CAT2(a, b) a##b
#define RT_CAT(a, b) RT_CAT2(a, b)

rt::KernelSlice RT_CAT(rt_kernel_slice_, RT_UNIT_NAME)()
{
    static const std::vector<rt::KernelEntry> entries = build_entries();
    return rt::KernelSlice{entries.data(), (int)entries.size()};
}
