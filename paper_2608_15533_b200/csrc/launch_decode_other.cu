// deltalog_decode_step, tiles other than 128 x 128: choice of the decode kernel and its launch.
#define DELTALOG_SHAPES_NOT_128
#include "launch_common.cuh"
#include "decode_kernel.cuh"
#include "decode_pipelined.cuh"
#include "decode_pipelined_d64.cuh"

namespace deltalog {
namespace {

// Tuning knobs (environment, read once): DELTALOG_DECODE_IMPL = 0 auto | 1 one-CTA-per-unit | 2 pipelined;
// DELTALOG_CTAS_PER_SM, DELTALOG_BASE_STAGES, DELTALOG_AUX_STAGES override the pipelined kernel's shape.

template <int OP, int DK, int DV, typename IO, typename UL, typename BT>
int launch_decode(const StateArgs &st_in, const TokenArgs &tk, cudaStream_t stream) {
    StateArgs st = st_in;
    const int total_units = tk.B * st.H;
    // The persistent kernels are built for square tiles (head size 128, and 64 with an fp32 base); other
    // shapes (d_k != d_v) run one CTA per unit.
    if constexpr (DK == DV) {
    constexpr int D = DK;
    static const int impl = env_int("DELTALOG_DECODE_IMPL", 0);
    static const int env_ctas = env_int("DELTALOG_CTAS_PER_SM", 0);
    static const int env_base = env_int("DELTALOG_BASE_STAGES", 0);
    static const int env_aux = env_int("DELTALOG_AUX_STAGES", 0);
    const DeviceInfo &dev = device_info();
    const int total = tk.B * st.H;

    // The pipelined kernel moves the scalar decay snapshots with 16-byte bulk copies, which needs
    // every unit's snapshot row to start on a 16-byte boundary: cap % 4 == 0 for GDN.
    // Head size 64: a unit is a single 16 KiB chunk and the per-unit hand-overs of the pipeline cost
    // more than they hide, so the one-CTA-per-unit kernel is the faster one there (measured).
    bool pipelined = impl != 1 && dev.sms > 0 && (OpTraits<OP>::kVecDecay || st.cap % 4 == 0) && (D == 128 || (impl == 2 && sizeof(BT) == 2));
    constexpr int kStage = chunk_bytes<D, BT>();
    constexpr int kChunks = D * D * (int)sizeof(BT) / kStage;  // chunks per base tile
    // hand-over slots: two while the base tile's arrival sets the pace; with a 16-bit base the chain
    // prep -> stream -> epilogue is the longer one and four units are kept in flight
    static const int env_slots = env_int("DELTALOG_PIPE_SLOTS", 0);
    PipeCfg cfg{0, 0, env_slots == 4 ? 2 : env_slots == 2 ? 1 : (sizeof(BT) == 2 ? 2 : 1), -1};  // depths set below
#if DELTALOG_TEST_HOOKS
    cfg.test_drop_item = env_int_now("DELTALOG_TEST_DROP_ITEM", -1);
#endif
    int ctas = env_ctas > 0 ? env_ctas : 1;
    if (pipelined) {
        // Shared memory of a CTA: barriers, hand-over slots, the base ring (its place is fixed, so that its
        // producers can start at once) and the region of the aux ring, whose stages the kernel sizes by the
        // longest live log among the CTA's units.  The region must hold two stages in the worst case (logs one
        // short of full); the base ring takes what is left, up to the depth that saturates HBM (fp32 base:
        // 128 KiB in flight per SM; 16-bit base: units pass twice as fast, a somewhat shorter ring and more aux
        // stages).  Each chunk of a tile has its own producer warp, which refills a stage as soon as THAT chunk
        // has been consumed; a warp's successive chunks are kChunks apart in the ring, so with fewer than kChunks
        // stages it would wait for a phase of the stage's barrier that it cannot tell from the one before
        // (one-bit parity): the ring must hold at least one whole tile, otherwise one CTA per unit it is.
        const int worst = 2 * AuxLayout<OP, D, IO, UL>(st.cap).bytes;
        const int fixed = kPipeBarrierBytes + pipe_scratch_bytes<D>(cfg.slot_shift);
        const bool b16 = sizeof(BT) == 2;
        int want_base = env_base > 0 ? env_base : (b16 ? 5 : 8) * (kChunkBytes / kStage);
        if (want_base < kChunks) want_base = kChunks;
        if (want_base > kPipeMaxBase) want_base = kPipeMaxBase;
        const int min_aux = env_aux > 0 ? env_aux : (b16 ? 6 : 4);   // aux stages wanted at the full capacity ...
        for (; ctas >= 1; --ctas) {
            int budget = dev.smem_per_sm / ctas - 1024;
            if (budget > dev.smem_optin) budget = dev.smem_optin;
            // ... as long as the base ring keeps its depth; at least the two stages of the worst case
            int aux_want = min_aux * (worst / 2);
            if (aux_want > budget - fixed - want_base * kStage) aux_want = budget - fixed - want_base * kStage;
            if (aux_want < worst) aux_want = worst;
            cfg.n_base = (budget - fixed - aux_want) / kStage;
            if (cfg.n_base > want_base) cfg.n_base = want_base;
            if (cfg.n_base >= kChunks) {
                cfg.aux_bytes = (budget - fixed - cfg.n_base * kStage) / 128 * 128;
                break;
            }
        }
        if (ctas < 1) pipelined = false;
    }
    if (pipelined) {
        // What L2 holds on to across steps is about half its size on this part (measured: a re-read set is
        // served in full up to 40-60 MB and not at all from ~100 MB on).  The log comes first; where the
        // full log leaves room, a fraction of the base tiles is asked to stay as well (config 1: 24 MB,
        // 2-3 % per step; with more, log and tiles push each other out).  DELTALOG_L2_PIN_MB overrides.
        static const int pin_mb = env_int("DELTALOG_L2_PIN_MB", -1);
        constexpr float kMiB = 1048576.f;
        const float entry = (float)(D * (sizeof(IO) + sizeof(UL)) + (OpTraits<OP>::kVecDecay ? D : 1) * 4);
        const float full_log = (float)total * (float)st.cap * entry;
        st.l2_pin_bytes = pin_mb >= 0 ? pin_mb * kMiB : fminf(24.f * kMiB, fmaxf(0.f, 64.f * kMiB - 0.75f * full_log));
        auto kernel = decode_pipelined_kernel<OP, D, IO, UL, BT>;
        const int smem = pipe_smem_bytes<D, BT>(cfg);
        if (int rc = ensure_smem(kernel, smem)) return rc;
        const int grid = total < dev.sms * ctas ? total : dev.sms * ctas;
        if (tk.hints & DELTALOG_HINT_BASE_UNTOUCHED) return launch_chained(kernel, grid, kPipeThreads, smem, stream, st, tk, cfg);
        kernel<<<grid, kPipeThreads, smem, stream>>>(st, tk, cfg);
        return finish_launch();
    }
    if constexpr (D == kP64D && std::is_same<BT, float>::value) {
        // Head size 64, fp32 base: the persistent kernel with warp-per-unit roles, whose operand stages are sized by
        // the live log length inside the kernel.  It needs room for at least four stages of each ring at the full capacity
        // beside the 8-tile base ring (always true up to capacity 32 or so), and 16-byte aligned snapshot rows.
        static const int env_aux_kb = env_int("DELTALOG_P64_AUX_KB", 0);
        P64Cfg c64{8, 8, 0};
        const int budget = (dev.smem_optin < dev.smem_per_sm - 1024 ? dev.smem_optin : dev.smem_per_sm - 1024);
        c64.aux_bytes = (budget - p64_smem_bytes(c64)) / 128 * 128;
        if (env_aux_kb > 0 && env_aux_kb * 1024 < c64.aux_bytes) c64.aux_bytes = env_aux_kb * 1024;
        const bool fits = c64.aux_bytes >= 4 * (KeyStage<OP, IO>(st.cap).bytes + ValStage<IO, UL>(st.cap).bytes);
        // Beyond 16 live entries the stages get so large that fewer than eight units are in flight and the
        // one-CTA-per-unit kernel is the faster one (measured on configuration 3's shape at capacity 32:
        // 105 - 144 us per launch against ~80 - 95 us from 17 entries on), so it keeps the larger capacities.
        static const int max_cap = env_int("DELTALOG_P64_MAX_CAP", 16);
        if (impl != 1 && dev.sms > 0 && fits && st.cap <= max_cap && st.cap <= kP64MaxCap &&
            (OpTraits<OP>::kVecDecay || st.cap % 4 == 0)) {
            auto kernel = decode_pipelined_d64_kernel<OP, IO, UL>;
            const int smem = p64_smem_bytes(c64);
            if (int rc = ensure_smem(kernel, smem)) return rc;
            const int grid = total < dev.sms ? total : dev.sms;
            if (tk.hints & DELTALOG_HINT_BASE_UNTOUCHED) return launch_chained(kernel, grid, kP64Threads, smem, stream, st, tk, c64);
            kernel<<<grid, kP64Threads, smem, stream>>>(st, tk, c64);
            return finish_launch();
        }
    }
    }
    auto kernel = decode_append_kernel<OP, DK, DV, IO, UL, BT>;
    const size_t smem = decode_smem_bytes<DK, DV, IO, UL>(OP, st.cap);
    if (int rc = ensure_smem(kernel, smem)) return rc;
    if (tk.hints & DELTALOG_HINT_BASE_UNTOUCHED)
        return launch_chained(kernel, total_units, decode_threads<DK, DV>(), smem, stream, st, tk);
    kernel<<<total_units, decode_threads<DK, DV>(), smem, stream>>>(st, tk);
    return finish_launch();
}


}  // namespace

int dispatch_decode_other(const deltalog_desc *desc, const StateArgs &st, const TokenArgs &tk, cudaStream_t s) {
#define CALL_DECODE(OP, DK, DV, IO) DELTALOG_WITH_UL(OP, IO, desc, launch_decode, DK, DV, st, tk, s)
    DELTALOG_DISPATCH(desc, CALL_DECODE);
#undef CALL_DECODE
    return DELTALOG_ERR_UNSUPPORTED_SHAPE;
}
}  // namespace deltalog
