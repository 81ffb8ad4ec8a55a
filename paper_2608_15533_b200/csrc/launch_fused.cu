// deltalog_decode_merge_step: the fused merge step.
#include "launch_common.cuh"
#include "fused_step_kernel.cuh"
#include "fused_step_resident.cuh"

namespace deltalog {
namespace {

template <int OP, int DK, int DV, typename IO, typename UL, typename BT>
int launch_fused_step(const StateArgs &st, const TokenArgs &tk, cudaStream_t stream) {
    // The resident kernel (the next unit's tile, log and token in flight while a unit is computed and stored) up to
    // capacity 16, where its shared memory leaves room for the same number of CTAs per SM as one unit per CTA has.
    // Its rank update costs more per live entry (scalar FMAs: 3.3 against 1.6 us per entry and launch on configuration
    // 1's shape), so one unit per CTA is the faster kernel beyond that (measured at capacity 8 / 16 / 24: 88 / 113 /
    // 140 us against 101 / 114 / 127 us; KDA shape at 16: 223 against 268 us; RWKV6 shape at 16 / 32: 125 / 181 against
    // 144 / 176 us).  DELTALOG_MAT_PREFETCH=0 keeps one unit per CTA everywhere.
    static const int prefetch = env_int("DELTALOG_MAT_PREFETCH", 1);
    const DeviceInfo &dev = device_info();
    if (prefetch && dev.sms > 0 && st.cap <= 16 && (OpTraits<OP>::kVecDecay || st.cap % 4 == 0)) {
        auto kernel = fused_step_resident_kernel<OP, DK, DV, IO, UL, BT>;
        const size_t bytes = FusedResidentLayout<OP, DK, DV, IO, UL, BT>(st.cap).bytes;
        constexpr int kWant = mat_threads<DK, DV>() <= 128 ? 4 : 2;
        if (bytes <= (size_t)dev.smem_optin && ensure_smem(kernel, bytes) == DELTALOG_OK) {
            const int ctas = resident_ctas(kernel, mat_threads<DK, DV>(), bytes);
            if (ctas >= kWant) {
                const int pairs = tk.B * st.H;
                const int grid = pairs < ctas * dev.sms ? pairs : ctas * dev.sms;
                int drop = -1;  // test builds only: the pair whose tile is never requested
#if DELTALOG_TEST_HOOKS
                drop = env_int_now("DELTALOG_TEST_DROP_ITEM", -1);
#endif
                kernel<<<grid, mat_threads<DK, DV>(), bytes, stream>>>(st, tk, pairs, drop);
                return finish_launch();
            }
        }
    }
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
