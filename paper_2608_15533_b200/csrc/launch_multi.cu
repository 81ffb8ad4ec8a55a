// deltalog_decode_steps: blocks of tokens.
#include "launch_common.cuh"
#include "decode_kernel.cuh"
#include "decode_multi_kernel.cuh"

namespace deltalog {
namespace {

template <int OP, int DK, int DV, typename IO, typename UL, typename BT>
int launch_decode_multi(const StateArgs &st, const TokenArgs &tk, int32_t T, cudaStream_t stream) {
    auto kernel = decode_multi_kernel<OP, DK, DV, IO, UL, BT>;
    const size_t smem = decode_smem_bytes<DK, DV, IO, UL>(OP, st.cap);
    if (int rc = ensure_smem(kernel, smem)) return rc;
    kernel<<<tk.B * st.H, decode_threads<DK, DV>(), smem, stream>>>(st, tk, T);
    return finish_launch();
}


}  // namespace

int dispatch_decode_multi(const deltalog_desc *desc, const StateArgs &st, const TokenArgs &tk, int32_t T, cudaStream_t s) {
#define CALL_MULTI(OP, DK, DV, IO) DELTALOG_WITH_UL(OP, IO, desc, launch_decode_multi, DK, DV, st, tk, T, s)
    DELTALOG_DISPATCH(desc, CALL_MULTI);
#undef CALL_MULTI
    return DELTALOG_ERR_UNSUPPORTED_SHAPE;
}
}  // namespace deltalog
