// deltalog_decode_merge_step: the fused merge step.
#include "launch_common.cuh"
#include "fused_step_kernel.cuh"

namespace deltalog {
namespace {

template <int OP, int DK, int DV, typename IO, typename UL, typename BT>
int launch_fused_step(const StateArgs &st, const TokenArgs &tk, cudaStream_t stream) {
    auto kernel = decode_merge_step_kernel<OP, DK, DV, IO, UL, BT>;
    const size_t smem = fused_step_smem_bytes<DK, DV, IO, UL>(st.cap, OpTraits<OP>::kVecDecay);
    if (int rc = ensure_smem(kernel, smem)) return rc;
    kernel<<<tk.B * st.H, mat_threads<DK, DV>(), smem, stream>>>(st, tk);
    return finish_launch();
}


}  // namespace

int dispatch_fused_step(const deltalog_desc *desc, const StateArgs &st, const TokenArgs &tk, cudaStream_t s) {
#define CALL_FUSED(OP, DK, DV, IO) DELTALOG_WITH_UL(OP, IO, desc, launch_fused_step, DK, DV, st, tk, s)
    DELTALOG_DISPATCH(desc, CALL_FUSED);
#undef CALL_FUSED
    return DELTALOG_ERR_UNSUPPORTED_SHAPE;
}
}  // namespace deltalog
