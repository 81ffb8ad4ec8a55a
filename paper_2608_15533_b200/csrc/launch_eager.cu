// deltalog_eager_step: the eager dense comparator.
#include "launch_common.cuh"
#include "eager_kernel.cuh"

namespace deltalog {
namespace {

template <int OP, int DK, int DV, typename IO>
int launch_eager(void *S, const deltalog_desc *d, int32_t *status, const TokenArgs &tk, cudaStream_t stream) {
    if constexpr (!std::is_same<IO, float>::value) {
        if (d->base_dtype == DELTALOG_BF16) {
            eager_step_kernel<OP, DK, DV, IO, __nv_bfloat16>
                <<<tk.B * d->H, kThreads, 0, stream>>>(S, d->num_slots, d->H, d->scale, status, tk);
            return finish_launch();
        }
    }
    eager_step_kernel<OP, DK, DV, IO, float><<<tk.B * d->H, kThreads, 0, stream>>>(S, d->num_slots, d->H, d->scale, status, tk);
    return finish_launch();
}


}  // namespace

int dispatch_eager(const deltalog_desc *desc, void *S, int32_t *status, const TokenArgs &tk, cudaStream_t s) {
#define CALL_EAGER(OP, DK, DV, IO) return launch_eager<OP, DK, DV, IO>(S, desc, status, tk, s)
    DELTALOG_DISPATCH(desc, CALL_EAGER);
#undef CALL_EAGER
    return DELTALOG_ERR_UNSUPPORTED_SHAPE;
}
}  // namespace deltalog
