// deltalog_merge and deltalog_reset_slots.
#include "launch_common.cuh"
#include "merge_kernel.cuh"
#include "merge_tc_kernel.cuh"

namespace deltalog {
namespace {

template <int OP, int DK, int DV, typename IO, typename UL, typename BT>
int launch_merge(const StateArgs &st, const int32_t *slot_idx, int32_t n, int32_t only_if_full,
                 cudaStream_t stream) {
    // DELTALOG_MERGE_TC = 1 (head size 128, no predicate): the contraction over the log entries runs
    // on the tensor cores (tcgen05, tf32 x 3).  Off by default: it executes a fraction of the
    // instructions, but with one unit per CTA the extra hand-overs (raw entries -> operands -> MMA ->
    // tensor-memory load) lengthen each CTA's dependent chain by more than the fp32 pipe costs
    // (measured on configuration 1: 110 / 119 / 142 / 215 us at capacity 4 / 16 / 32 / 64 against
    // 85 / 99 / 130 / 195 us for the packed-FMA kernel).
    static const int use_tc = env_int("DELTALOG_MERGE_TC", 0);
    if constexpr (DK == kTcD && DV == kTcD && std::is_same<BT, float>::value) {
        if (use_tc && !only_if_full) {
            auto kernel = merge_tc_kernel<OP, IO, UL>;
            const size_t bytes = merge_tc_smem_bytes<OP, IO, UL>(st.cap);
            if (int rc = ensure_smem(kernel, bytes)) return rc;
            kernel<<<n * st.H, kThreads, bytes, stream>>>(st, slot_idx, only_if_full);
            return finish_launch();
        }
    }
    const size_t smem = merge_smem_bytes<DK, DV, IO, UL>(st.cap, OpTraits<OP>::kVecDecay);
    // Without the predicate every listed unit is expected to fold: one unit per CTA.  With it (one
    // call over a whole batch whose fills are staggered) most units are skipped: kMergePack candidates per CTA.
    const int pairs = n * st.H;
    if (only_if_full) {
        auto kernel = merge_kernel<OP, DK, DV, IO, UL, kMergePack, BT>;
        if (int rc = ensure_smem(kernel, smem)) return rc;
        kernel<<<(pairs + kMergePack - 1) / kMergePack, mat_threads<DK, DV>(), smem, stream>>>(st, slot_idx, only_if_full, pairs);
    } else {
        auto kernel = merge_kernel<OP, DK, DV, IO, UL, 1, BT>;
        if (int rc = ensure_smem(kernel, smem)) return rc;
        kernel<<<pairs, mat_threads<DK, DV>(), smem, stream>>>(st, slot_idx, only_if_full, pairs);
    }
    return finish_launch();
}


}  // namespace

int dispatch_merge(const deltalog_desc *desc, const StateArgs &st, const int32_t *slot_idx, int32_t n, int32_t only_if_full,
                   cudaStream_t s) {
#define CALL_MERGE(OP, DK, DV, IO) DELTALOG_WITH_UL(OP, IO, desc, launch_merge, DK, DV, st, slot_idx, n, only_if_full, s)
    DELTALOG_DISPATCH(desc, CALL_MERGE);
#undef CALL_MERGE
    return DELTALOG_ERR_UNSUPPORTED_SHAPE;
}

int dispatch_reset_slots(const deltalog_desc *desc, const StateArgs &st, const int32_t *slot_idx, int32_t n, const float *S_init,
                         cudaStream_t s) {
    const int tile = desc->d_k * desc->d_v;
    if (desc->base_dtype == DELTALOG_BF16) reset_slots_kernel<__nv_bfloat16><<<n * st.H, kThreads, 0, s>>>(st, slot_idx, S_init, tile);
    else reset_slots_kernel<float><<<n * st.H, kThreads, 0, s>>>(st, slot_idx, S_init, tile);
    return finish_launch();
}
}  // namespace deltalog
