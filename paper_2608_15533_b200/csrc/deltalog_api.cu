// C ABI of the DeltaLog decode library: host-side argument validation and kernel dispatch.
// Declarations and the contract of every entry point are in include/deltalog.h.
#include <atomic>
#include <map>
#include <mutex>
#include <utility>
#include <cstdint>
#include <type_traits>

#include <cstdlib>

#include "decode_kernel.cuh"
#include "decode_multi_kernel.cuh"
#include "decode_pipelined.cuh"
#include "decode_pipelined_d64.cuh"
#include "eager_kernel.cuh"
#include "fused_step_kernel.cuh"
#include "merge_kernel.cuh"
#include "merge_tc_kernel.cuh"
#include "validate.h"

namespace deltalog {
namespace {

std::atomic<uint64_t> g_launches{0};

int qk_heads(const deltalog_desc *d) { return d->H_qk > 0 ? d->H_qk : d->H; }

TokenArgs make_token_args(const deltalog_desc *d, const void *q, const void *k, const void *v, const float *g,
                          const float *beta, const float *u_bonus, const int32_t *slot_idx, void *out, int32_t B) {
    // plain linear attention has no gate: the kernels see a null pointer and use lambda = 0
    return TokenArgs{q, k, v, op_has_gate(d->op) ? g : nullptr, beta, u_bonus, slot_idx, out, B, qk_heads(d), d->H / qk_heads(d),
                     d->hints};
}

size_t round256(size_t x) { return (x + 255) / 256 * 256; }

// Host and staging buffers are "packed" when q, k, v, g (if the operator has a gate) and beta (delta
// rule) follow one another in this order, each starting on the next 256-byte boundary after the
// previous one ends, on BOTH sides: the five copies then collapse into one over the whole block.
// Returns the block's size, or 0 when the layout is not packed.
size_t packed_block_bytes(const deltalog_desc *d, const deltalog_staging *stg, const void *hq, const void *hk,
                          const void *hv, const float *hg, const float *hbeta, size_t qk_vec, size_t vec,
                          size_t gbytes, size_t units) {
    if (!stg->packed) return 0;  // adjacency alone proves nothing: the block must be one allocation
    const char *h = static_cast<const char *>(hq);
    const char *s = static_cast<const char *>(stg->q);
    size_t off = round256(qk_vec);
    if (static_cast<const char *>(hk) != h + off || static_cast<const char *>(stg->k) != s + off) return 0;
    off += round256(qk_vec);
    if (static_cast<const char *>(hv) != h + off || static_cast<const char *>(stg->v) != s + off) return 0;
    size_t end = off + vec;
    off += round256(vec);
    if (op_has_gate(d->op)) {
        if (reinterpret_cast<const char *>(hg) != h + off || reinterpret_cast<const char *>(stg->g) != s + off) return 0;
        end = off + gbytes;
        off += round256(gbytes);
    }
    if (op_delta_rule(d->op)) {
        if (reinterpret_cast<const char *>(hbeta) != h + off || reinterpret_cast<const char *>(stg->beta) != s + off) return 0;
        end = off + units * sizeof(float);
    }
    return end;
}

int env_int(const char *name, int dflt) {
    const char *v = std::getenv(name);
    return v ? std::atoi(v) : dflt;
}
#if DELTALOG_TEST_HOOKS
int env_int_now(const char *name, int dflt) { return env_int(name, dflt); }  // read at every launch
#endif

StateArgs make_state_args(const deltalog_desc *d, const deltalog_state *s) {
    StateArgs a;
    a.S_base = s->S_base;
    a.K_log = s->K_log;
    a.U_log = s->U_log;
    a.decay_log = s->decay_log;
    a.log_len = s->log_len;
    a.status = s->status;
    a.num_slots = d->num_slots;
    a.H = d->H;
    a.cap = d->cap;
    a.scale = d->scale;
    static const int keep_mb = env_int("DELTALOG_L2_KEEP_MB", 40);
    a.l2_keep_bytes = (float)keep_mb * 1048576.f;
    a.l2_pin_bytes = 0.f;  // set per launch by the pipelined decode kernel's launcher
    return a;
}

int finish_launch() {
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? DELTALOG_OK : DELTALOG_ERR_CUDA;
}

// Raise the dynamic shared-memory limit of a kernel when a launch needs more than 48 KiB.  The limit
// only ever grows (per device), and it is raised to what launches have asked for, not to the device
// maximum: a kernel with static shared memory cannot be granted the whole opt-in size as dynamic.
template <typename K>
int ensure_smem(K kernel, size_t bytes) {
    if (bytes <= 48 * 1024) return DELTALOG_OK;
    static std::mutex mu;
    static std::map<std::pair<int, const void *>, size_t> granted;  // (device, kernel) -> bytes granted
    int dev = 0;
    cudaGetDevice(&dev);
    const auto key = std::make_pair(dev, reinterpret_cast<const void *>(kernel));
    std::lock_guard<std::mutex> lock(mu);
    size_t &g = granted[key];
    if (bytes <= g) return DELTALOG_OK;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) {
        cudaGetLastError();  // not sticky: leave the runtime clean for the caller
        return DELTALOG_ERR_CUDA;
    }
    g = bytes;
    return DELTALOG_OK;
}

// Launch with programmatic stream serialisation: the caller promised (DELTALOG_HINT_BASE_UNTOUCHED) that
// the kernel in front of this one on the stream does not write this state's base tiles, so this
// kernel's CTAs may start, and request base tiles, while that kernel is still retiring.
template <typename K, typename... Args>
int launch_chained(K kernel, int grid, int threads, size_t smem, cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(grid);
    lc.blockDim = dim3(threads);
    lc.dynamicSmemBytes = smem;
    lc.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    if (cudaLaunchKernelEx(&lc, kernel, args...) != cudaSuccess) {
        cudaGetLastError();
        return DELTALOG_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return DELTALOG_OK;
}

// Device facts needed to size the persistent kernel, queried once per device.
struct DeviceInfo {
    int sms = 0;
    int smem_per_sm = 0;
    int smem_optin = 0;
};
const DeviceInfo &device_info() {
    static DeviceInfo info[64];
    int dev = 0;
    cudaGetDevice(&dev);
    DeviceInfo &d = info[dev & 63];
    if (d.sms == 0) {
        cudaDeviceGetAttribute(&d.smem_per_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev);
        cudaDeviceGetAttribute(&d.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
        cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev);
    }
    return d;
}

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
        if (impl != 1 && dev.sms > 0 && fits && st.cap <= max_cap && (OpTraits<OP>::kVecDecay || st.cap % 4 == 0)) {
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

template <int OP, int DK, int DV, typename IO, typename UL, typename BT>
int launch_decode_multi(const StateArgs &st, const TokenArgs &tk, int32_t T, cudaStream_t stream) {
    auto kernel = decode_multi_kernel<OP, DK, DV, IO, UL, BT>;
    const size_t smem = decode_smem_bytes<DK, DV, IO, UL>(OP, st.cap);
    if (int rc = ensure_smem(kernel, smem)) return rc;
    kernel<<<tk.B * st.H, decode_threads<DK, DV>(), smem, stream>>>(st, tk, T);
    return finish_launch();
}

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
    const size_t smem = merge_smem_bytes<DK, DV>(st.cap);
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

template <int OP, int DK, int DV, typename IO, typename UL, typename BT>
int launch_fused_step(const StateArgs &st, const TokenArgs &tk, cudaStream_t stream) {
    auto kernel = decode_merge_step_kernel<OP, DK, DV, IO, UL, BT>;
    const size_t smem = fused_step_smem_bytes<DK, DV>(st.cap);
    if (int rc = ensure_smem(kernel, smem)) return rc;
    kernel<<<tk.B * st.H, mat_threads<DK, DV>(), smem, stream>>>(st, tk);
    return finish_launch();
}

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

// Expand (op, d_k, d_v, io dtype) into the template instantiation: CALL(OP, DK, DV, IO).
#define DELTALOG_DISPATCH(desc, CALL)                                                        \
    do {                                                                                     \
        const int op_ = (desc)->op, dk_ = (desc)->d_k, dv_ = (desc)->d_v, io_ = (desc)->io_dtype; \
        if (op_ == DELTALOG_GDN) {                                                           \
            DELTALOG_DISPATCH_D(DELTALOG_GDN, dk_, dv_, io_, CALL);                          \
        } else if (op_ == DELTALOG_KDA) {                                                    \
            DELTALOG_DISPATCH_D(DELTALOG_KDA, dk_, dv_, io_, CALL);                          \
        } else if (op_ == DELTALOG_RETNET || op_ == DELTALOG_LINATTN) {                      \
            DELTALOG_DISPATCH_D(DELTALOG_RETNET, dk_, dv_, io_, CALL); /* linear attention: null gate */ \
        } else if (op_ == DELTALOG_GLA) {                                                    \
            DELTALOG_DISPATCH_D(DELTALOG_GLA, dk_, dv_, io_, CALL);                          \
        } else {                                                                             \
            DELTALOG_DISPATCH_D(DELTALOG_RWKV6, dk_, dv_, io_, CALL);                        \
        }                                                                                    \
    } while (0)
#define DELTALOG_DISPATCH_D(OP, dk_, dv_, io_, CALL)                                         \
    if (dk_ == 64 && dv_ == 64) {                                                            \
        DELTALOG_DISPATCH_IO(OP, 64, 64, io_, CALL);                                         \
    } else if (dk_ == 128 && dv_ == 128) {                                                   \
        DELTALOG_DISPATCH_IO(OP, 128, 128, io_, CALL);                                       \
    } else if (dk_ == 128) {                                                                 \
        DELTALOG_DISPATCH_IO(OP, 128, 64, io_, CALL);                                        \
    } else {                                                                                 \
        DELTALOG_DISPATCH_IO(OP, 64, 128, io_, CALL);                                        \
    }
#define DELTALOG_DISPATCH_IO(OP, DK, DV, io_, CALL)                                          \
    if (io_ == DELTALOG_F32) { CALL(OP, DK, DV, float); } else { CALL(OP, DK, DV, __nv_bfloat16); }

// The value-side log keeps the I/O dtype where b = v (lossless).  For the delta rule it is fp32 by
// default; a 16-bit U log (descriptor ulog_dtype == io_dtype == BF16) is the reduced-precision variant.
// The dense base is fp32 unless the descriptor asks for the 16-bit state (16-bit I/O only).
#define DELTALOG_WITH_UL(OP, IO, desc, FN, DK, DV, ...)                                                    \
    do {                                                                                                  \
        if constexpr (!std::is_same<IO, float>::value) {                                                  \
            if ((desc)->base_dtype == DELTALOG_BF16) {                                                    \
                DELTALOG_WITH_UL_BT(OP, IO, __nv_bfloat16, desc, FN, DK, DV, __VA_ARGS__);                \
            }                                                                                             \
        }                                                                                                 \
        DELTALOG_WITH_UL_BT(OP, IO, float, desc, FN, DK, DV, __VA_ARGS__);                                 \
    } while (0)
#define DELTALOG_WITH_UL_BT(OP, IO, BT, desc, FN, DK, DV, ...)                                             \
    do {                                                                                                  \
        if constexpr (OpTraits<OP>::kDeltaRule) {                                                         \
            if constexpr (!std::is_same<IO, float>::value) {                                              \
                if ((desc)->ulog_dtype != DELTALOG_F32) return FN<OP, DK, DV, IO, IO, BT>(__VA_ARGS__);    \
            }                                                                                             \
            return FN<OP, DK, DV, IO, float, BT>(__VA_ARGS__);                                            \
        } else {                                                                                          \
            return FN<OP, DK, DV, IO, IO, BT>(__VA_ARGS__);                                               \
        }                                                                                                 \
    } while (0)

}  // namespace
}  // namespace deltalog

using namespace deltalog;

extern "C" {

int deltalog_decode_step(const deltalog_desc *desc, const deltalog_state *state, const void *q,
                         const void *k, const void *v, const float *g, const float *beta,
                         const float *u_bonus, const int32_t *slot_idx, int32_t B, void *out,
                         void *stream) {
    if (int rc = validate_desc(desc)) return rc;
    if (int rc = validate_state(state)) return rc;
    if (int rc = validate_token(desc, q, k, v, g, beta, u_bonus, B, out)) return rc;
    if (B == 0) return DELTALOG_OK;
    const StateArgs st = make_state_args(desc, state);
    const TokenArgs tk = make_token_args(desc, q, k, v, g, beta, u_bonus, slot_idx, out, B);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
#define CALL_DECODE(OP, DK, DV, IO) DELTALOG_WITH_UL(OP, IO, desc, launch_decode, DK, DV, st, tk, s)
    DELTALOG_DISPATCH(desc, CALL_DECODE);
#undef CALL_DECODE
    return DELTALOG_ERR_INVALID_ARG;
}

int deltalog_decode_steps(const deltalog_desc *desc, const deltalog_state *state, const void *q, const void *k,
                          const void *v, const float *g, const float *beta, const float *u_bonus,
                          const int32_t *slot_idx, int32_t B, int32_t T, void *out, void *stream) {
    if (int rc = validate_desc(desc)) return rc;
    if (int rc = validate_state(state)) return rc;
    if (int rc = validate_token(desc, q, k, v, g, beta, u_bonus, B, out)) return rc;
    if (T < 1 || T > desc->cap) return DELTALOG_ERR_CAP_RANGE;
    if (B == 0) return DELTALOG_OK;
    const StateArgs st = make_state_args(desc, state);
    const TokenArgs tk = make_token_args(desc, q, k, v, g, beta, u_bonus, slot_idx, out, B);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
#define CALL_MULTI(OP, DK, DV, IO) DELTALOG_WITH_UL(OP, IO, desc, launch_decode_multi, DK, DV, st, tk, T, s)
    DELTALOG_DISPATCH(desc, CALL_MULTI);
#undef CALL_MULTI
    return DELTALOG_ERR_INVALID_ARG;
}

int deltalog_decode_merge_step(const deltalog_desc *desc, const deltalog_state *state, const void *q,
                               const void *k, const void *v, const float *g, const float *beta,
                               const float *u_bonus, const int32_t *slot_idx, int32_t B, void *out,
                               void *stream) {
    if (int rc = validate_desc(desc)) return rc;
    if (int rc = validate_state(state)) return rc;
    if (int rc = validate_token(desc, q, k, v, g, beta, u_bonus, B, out)) return rc;
    if (B == 0) return DELTALOG_OK;
    const StateArgs st = make_state_args(desc, state);
    const TokenArgs tk = make_token_args(desc, q, k, v, g, beta, u_bonus, slot_idx, out, B);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
#define CALL_FUSED(OP, DK, DV, IO) DELTALOG_WITH_UL(OP, IO, desc, launch_fused_step, DK, DV, st, tk, s)
    DELTALOG_DISPATCH(desc, CALL_FUSED);
#undef CALL_FUSED
    return DELTALOG_ERR_INVALID_ARG;
}

int deltalog_merge(const deltalog_desc *desc, const deltalog_state *state, const int32_t *slot_idx,
                   int32_t n, int32_t only_if_full, void *stream) {
    if (int rc = validate_desc(desc)) return rc;
    if (int rc = validate_state(state)) return rc;
    if (n < 0 || (!slot_idx && n > desc->num_slots)) return DELTALOG_ERR_INVALID_ARG;
    if (n == 0) return DELTALOG_OK;
    const StateArgs st = make_state_args(desc, state);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
#define CALL_MERGE(OP, DK, DV, IO) DELTALOG_WITH_UL(OP, IO, desc, launch_merge, DK, DV, st, slot_idx, n, only_if_full, s)
    DELTALOG_DISPATCH(desc, CALL_MERGE);
#undef CALL_MERGE
    return DELTALOG_ERR_INVALID_ARG;
}

int deltalog_reset_slots(const deltalog_desc *desc, const deltalog_state *state, const int32_t *slot_idx,
                         int32_t n, const float *S_init, void *stream) {
    if (int rc = validate_desc(desc)) return rc;
    if (int rc = validate_state(state)) return rc;
    if (n < 0 || (!slot_idx && n > desc->num_slots) || (S_init && !aligned16(S_init))) return DELTALOG_ERR_INVALID_ARG;
    if (n == 0) return DELTALOG_OK;
    const StateArgs st = make_state_args(desc, state);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const bool b16 = desc->base_dtype == DELTALOG_BF16;
    const int tile = desc->d_k * desc->d_v;
    if (b16) reset_slots_kernel<__nv_bfloat16><<<n * st.H, kThreads, 0, s>>>(st, slot_idx, S_init, tile);
    else reset_slots_kernel<float><<<n * st.H, kThreads, 0, s>>>(st, slot_idx, S_init, tile);
    return finish_launch();
}

int deltalog_eager_step(const deltalog_desc *desc, void *S, const void *q, const void *k,
                        const void *v, const float *g, const float *beta, const float *u_bonus,
                        const int32_t *slot_idx, int32_t B, void *out, int32_t *status, void *stream) {
    if (int rc = validate_desc(desc)) return rc;
    if (!S || !aligned16(S)) return DELTALOG_ERR_INVALID_ARG;
    if (int rc = validate_token(desc, q, k, v, g, beta, u_bonus, B, out)) return rc;
    if (B == 0) return DELTALOG_OK;
    const TokenArgs tk = make_token_args(desc, q, k, v, g, beta, u_bonus, slot_idx, out, B);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
#define CALL_EAGER(OP, DK, DV, IO) return launch_eager<OP, DK, DV, IO>(S, desc, status, tk, s)
    DELTALOG_DISPATCH(desc, CALL_EAGER);
#undef CALL_EAGER
    return DELTALOG_ERR_INVALID_ARG;
}

int deltalog_decode_step_host(const deltalog_desc *desc, const deltalog_state *state,
                              const deltalog_staging *staging, const void *host_q,
                              const void *host_k, const void *host_v, const float *host_g,
                              const float *host_beta, const float *u_bonus,
                              const int32_t *slot_idx, int32_t B, void *host_out, void *stream) {
    // every check of the decode step runs before the first copy is enqueued: a rejected call leaves the
    // stream and the staging buffers as they were
    if (int rc = validate_desc(desc)) return rc;
    if (int rc = validate_state(state)) return rc;
    if (!staging || !host_q || !host_k || !host_v || !host_out) return DELTALOG_ERR_INVALID_ARG;
    if (op_has_gate(desc->op) && (!host_g || !staging->g)) return DELTALOG_ERR_INVALID_ARG;
    if (op_delta_rule(desc->op) && (!host_beta || !staging->beta)) return DELTALOG_ERR_INVALID_ARG;
    if (int rc = validate_token(desc, staging->q, staging->k, staging->v, staging->g, staging->beta, u_bonus, B, staging->out))
        return rc;
    if (B == 0) return DELTALOG_OK;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t units = (size_t)B * desc->H;
    const size_t esz = desc->io_dtype == DELTALOG_F32 ? 4 : 2;
    const size_t vec = units * desc->d_v * esz;
    const size_t qk_vec = (size_t)B * qk_heads(desc) * desc->d_k * esz;
    const size_t gbytes = units * (op_vec_decay(desc->op) ? desc->d_k : 1) * sizeof(float);
    bool ok = true;
    if (const size_t block = packed_block_bytes(desc, staging, host_q, host_k, host_v, host_g, host_beta, qk_vec, vec,
                                                gbytes, units)) {
        ok = cudaMemcpyAsync(staging->q, host_q, block, cudaMemcpyHostToDevice, s) == cudaSuccess;  // one copy
    } else {
        ok = cudaMemcpyAsync(staging->q, host_q, qk_vec, cudaMemcpyHostToDevice, s) == cudaSuccess;
        ok = ok && cudaMemcpyAsync(staging->k, host_k, qk_vec, cudaMemcpyHostToDevice, s) == cudaSuccess;
        ok = ok && cudaMemcpyAsync(staging->v, host_v, vec, cudaMemcpyHostToDevice, s) == cudaSuccess;
        if (op_has_gate(desc->op))
            ok = ok && cudaMemcpyAsync(staging->g, host_g, gbytes, cudaMemcpyHostToDevice, s) == cudaSuccess;
        if (op_delta_rule(desc->op))
            ok = ok && cudaMemcpyAsync(staging->beta, host_beta, units * sizeof(float), cudaMemcpyHostToDevice, s) ==
                           cudaSuccess;
    }
    if (!ok) return DELTALOG_ERR_CUDA;
    if (int rc = deltalog_decode_step(desc, state, staging->q, staging->k, staging->v, staging->g,
                                      staging->beta, u_bonus, slot_idx, B, staging->out, stream))
        return rc;
    if (cudaMemcpyAsync(host_out, staging->out, units * desc->d_v * esz, cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return DELTALOG_ERR_CUDA;
    return DELTALOG_OK;
}

int deltalog_decode_step_host_overlapped(const deltalog_desc *desc, const deltalog_state *state,
                                         const deltalog_staging *staging, const deltalog_host_lane *lane,
                                         const void *host_q, const void *host_k, const void *host_v,
                                         const float *host_g, const float *host_beta, const float *u_bonus,
                                         const int32_t *slot_idx, int32_t B, void *host_out) {
    if (int rc = validate_desc(desc)) return rc;
    if (int rc = validate_state(state)) return rc;
    if (!staging || !lane || !host_q || !host_k || !host_v || !host_out) return DELTALOG_ERR_INVALID_ARG;
    if (!lane->in_done || !lane->compute_done || !lane->out_done) return DELTALOG_ERR_INVALID_ARG;
    if (op_has_gate(desc->op) && (!host_g || !staging->g)) return DELTALOG_ERR_INVALID_ARG;
    if (op_delta_rule(desc->op) && (!host_beta || !staging->beta)) return DELTALOG_ERR_INVALID_ARG;
    if (int rc = validate_token(desc, staging->q, staging->k, staging->v, staging->g, staging->beta, u_bonus, B, staging->out))
        return rc;
    if (B == 0) return DELTALOG_OK;
    cudaStream_t s_in = static_cast<cudaStream_t>(lane->copy_in_stream);
    cudaStream_t s_cmp = static_cast<cudaStream_t>(lane->compute_stream);
    cudaStream_t s_out = static_cast<cudaStream_t>(lane->copy_out_stream);
    cudaEvent_t e_in = static_cast<cudaEvent_t>(lane->in_done);
    cudaEvent_t e_cmp = static_cast<cudaEvent_t>(lane->compute_done);
    cudaEvent_t e_out = static_cast<cudaEvent_t>(lane->out_done);
    const size_t units = (size_t)B * desc->H;
    const size_t esz = desc->io_dtype == DELTALOG_F32 ? 4 : 2;
    const size_t vec = units * desc->d_v * esz;
    const size_t qk_vec = (size_t)B * qk_heads(desc) * desc->d_k * esz;
    const size_t gbytes = units * (op_vec_decay(desc->op) ? desc->d_k : 1) * sizeof(float);
    // copy-in stream: the staging inputs are free once the kernel that last read them is done
    bool ok = cudaStreamWaitEvent(s_in, e_cmp, 0) == cudaSuccess;
    if (const size_t block = packed_block_bytes(desc, staging, host_q, host_k, host_v, host_g, host_beta, qk_vec, vec,
                                                gbytes, units)) {
        ok = ok && cudaMemcpyAsync(staging->q, host_q, block, cudaMemcpyHostToDevice, s_in) == cudaSuccess;  // one copy
    } else {
        ok = ok && cudaMemcpyAsync(staging->q, host_q, qk_vec, cudaMemcpyHostToDevice, s_in) == cudaSuccess;
        ok = ok && cudaMemcpyAsync(staging->k, host_k, qk_vec, cudaMemcpyHostToDevice, s_in) == cudaSuccess;
        ok = ok && cudaMemcpyAsync(staging->v, host_v, vec, cudaMemcpyHostToDevice, s_in) == cudaSuccess;
        if (op_has_gate(desc->op))
            ok = ok && cudaMemcpyAsync(staging->g, host_g, gbytes, cudaMemcpyHostToDevice, s_in) == cudaSuccess;
        if (op_delta_rule(desc->op))
            ok = ok && cudaMemcpyAsync(staging->beta, host_beta, units * sizeof(float), cudaMemcpyHostToDevice, s_in) ==
                           cudaSuccess;
    }
    ok = ok && cudaEventRecord(e_in, s_in) == cudaSuccess;
    // compute stream: inputs landed, and the previous output of this staging set has been read back
    ok = ok && cudaStreamWaitEvent(s_cmp, e_in, 0) == cudaSuccess;
    ok = ok && cudaStreamWaitEvent(s_cmp, e_out, 0) == cudaSuccess;
    if (!ok) return DELTALOG_ERR_CUDA;
    if (int rc = deltalog_decode_step(desc, state, staging->q, staging->k, staging->v, staging->g,
                                      staging->beta, u_bonus, slot_idx, B, staging->out, lane->compute_stream))
        return rc;
    ok = cudaEventRecord(e_cmp, s_cmp) == cudaSuccess;
    // copy-out stream
    ok = ok && cudaStreamWaitEvent(s_out, e_cmp, 0) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(host_out, staging->out, units * desc->d_v * esz, cudaMemcpyDeviceToHost, s_out) ==
                   cudaSuccess;
    ok = ok && cudaEventRecord(e_out, s_out) == cudaSuccess;
    return ok ? DELTALOG_OK : DELTALOG_ERR_CUDA;
}

const char *deltalog_status_string(int code) {
    switch (code) {
        case DELTALOG_OK: return "ok";
        case DELTALOG_ERR_INVALID_ARG: return "invalid argument (null / misaligned pointer, bad enum or negative count)";
        case DELTALOG_ERR_UNSUPPORTED_SHAPE: return "unsupported shape or dtype combination";
        case DELTALOG_ERR_CAP_RANGE: return "log capacity outside 1..64";
        case DELTALOG_ERR_CUDA: return "CUDA runtime error";
        case DELTALOG_ERR_STATIC_LIMIT: return "request larger than the built-in staging area (DELTALOG_STATIC_STAGING_BYTES)";
        default: return "unknown status code";
    }
}

int deltalog_version(void) { return 200; }

#ifndef DELTALOG_BUILD_ID
#define DELTALOG_BUILD_ID "unknown"
#endif
const char *deltalog_build_id(void) { return DELTALOG_BUILD_ID; }

uint64_t deltalog_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
