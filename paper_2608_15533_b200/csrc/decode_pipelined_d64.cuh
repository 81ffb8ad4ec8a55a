// Persistent, warp-specialised decode + append kernel for head size 64 (fp32 base).
//
// Same arithmetic as decode_append_kernel (Algorithm 1, append branch; Eq. 4 and Eq. 6).  At head
// size 64 a unit is one 16 KiB chunk of base plus a few KiB of log: what limits a pipeline here is the
// fixed cost per unit, not the bytes.  So the per-unit scalar work is spread over warps that each own
// a unit, several units are in flight at every stage, and the producers issue their copies from
// several warps side by side:
//
//   base producers (2 warps)  warp b brings the 16 KiB tiles of units b, b+2, ... (one bulk copy each);
//   aux producers  (4 warps)  warp a owns units a, a+4, ...: live K, U, Lambda entries, q, k, v, gate,
//                             bonus and a metadata record (one thread needs about a microsecond for a
//                             unit's copies, so several units are queued in parallel);
//   prep warps     (4 warps)  warp p owns units p, p+4, ...: cumulative decay, decayed multipliers
//                             (-> stream warps), key-side replay coefficients, q.k (-> epilogue);
//   stream warps   (4 warps)  warp w owns units w, w+4, ...: the base pass S_base^T (e^lbar . k) and
//                             S_base^T (e^lbar . q) over the whole 64 x 64 tile;
//   epilogue warps (4 warps)  warp e owns units e, e+4, ...: value-side replay, b, the output and the
//                             append.
//
// How many units an SM keeps in flight is set by the rings that hold a unit's small operands: a stage
// is occupied from the moment its copies are queued until its last reader is done, so a ring's depth
// divided by that time is the unit rate.  Two measures keep that rate above the rate of the tile
// stream.  (1) The operands travel in two rings with different life times: the key side (K, Lambda,
// q, k, gate, bonus -- three quarters of the bytes for per-key decay) is read by the prep warp only
// and released about 3 us after its copies were queued; the value side (U, v) waits for the stream
// and epilogue warps, about 5 us.  (2) The stages are sized by the longest LIVE log among the CTA's
// units, found in a short prologue (the base producers do not wait for it: the base ring has a fixed
// place), and the two depths are chosen for that size.  With one ring of stages sized for the full
// capacity only 8 units were in flight beside the 8-tile base ring -- the rate of the
// one-CTA-per-unit kernel.
//
// Ring depths are multiples of the number of warps that take turns waiting on a ring, so that a stage
// is always awaited by the same warp in program order (the one-bit phase parity of an mbarrier wait
// is ambiguous for a waiter that may be two phases off).  Hand-over through mbarriers and a ring of
// per-unit slots; every wait is bounded in time (DELTALOG_STATUS_TIMEOUT, never a hang).
#pragma once

#include "decode_pipelined.cuh"

namespace deltalog {

constexpr int kP64D = 64;
constexpr int kP64StreamWarps = 4;
constexpr int kP64AuxWarps = 4;
constexpr int kP64BaseWarps = 2;
constexpr int kP64MaxKey = 16;             // upper bounds on the depths of the key-side and value-side rings
constexpr int kP64MaxVal = 32;             // (mbarrier storage)
constexpr int kP64Threads = 32 * (kP64StreamWarps + 4 + 4 + kP64BaseWarps + kP64AuxWarps);  // stream, prep, epilogue, base and aux producers
constexpr int kP64ScalarWarps = 4;         // prep warps, and as many epilogue warps
constexpr int kP64BarrierBytes = 2048;
// hand-over slot (floats): q, k, mul_k, mul_q, lbar, lbar' [6 x 64], ck, cq [2 x kP64MaxCap], scalars [4],
// the two base-pass results [2][64]
constexpr int kP64MaxCap = 32;             // largest capacity this kernel takes (sizes the coefficient arrays of a slot)
constexpr int kP64SlotFloats = 6 * 64 + 2 * kP64MaxCap + 4 + 2 * 64;
constexpr int kP64SlotBytes = (kP64SlotFloats * 4 + 127) / 128 * 128;

// Byte offsets inside a key-side stage and a value-side stage with room for n log entries.
template <int OP, typename IO>
struct KeyStage {
    static constexpr bool kVec = OpTraits<OP>::kVecDecay;
    static constexpr int DL = kVec ? kP64D : 1;
    int K, L, q, k, g, bonus, meta, bytes;
    __host__ __device__ explicit KeyStage(int n) {
        K = 0;
        L = K + n * kP64D * (int)sizeof(IO);
        q = L + align_up(n * DL * 4, 16);
        k = q + kP64D * (int)sizeof(IO);
        g = k + kP64D * (int)sizeof(IO);
        bonus = g + (kVec ? kP64D * 4 : 0);
        meta = bonus + (OP == DELTALOG_RWKV6 ? kP64D * 4 : 0);
        bytes = align_up(meta + 32, 128);
    }
};
template <typename IO, typename UL>
struct ValStage {
    int U, v, meta, bytes;
    __host__ __device__ explicit ValStage(int n) {
        U = 0;
        v = U + n * kP64D * (int)sizeof(UL);
        meta = v + kP64D * (int)sizeof(IO);
        bytes = align_up(meta + 32, 128);
    }
};

struct P64Cfg {
    int n_base;     // stages of the base ring (one 16 KiB tile each), a multiple of 4
    int n_slots;    // hand-over slots, a multiple of 4
    int aux_bytes;  // bytes shared by the key-side and value-side rings; their depths follow from the live log lengths
};

__host__ inline int p64_smem_bytes(P64Cfg cfg) {
    return kP64BarrierBytes + cfg.n_slots * kP64SlotBytes + cfg.n_base * kChunkBytes + cfg.aux_bytes;
}

template <int OP, typename IO, typename UL>
__global__ void __launch_bounds__(kP64Threads, 1) decode_pipelined_d64_kernel(StateArgs st, TokenArgs tk, P64Cfg cfg) {
    constexpr int D = kP64D;
    constexpr bool kDelta = OpTraits<OP>::kDeltaRule;
    constexpr bool kPost = OpTraits<OP>::kPostReadout;
    constexpr bool kVecDecay = OpTraits<OP>::kVecDecay;
    constexpr int DL = kVecDecay ? D : 1;
    constexpr int oQ = 0, oK = 64, oMK = 128, oMQ = 192, oLB = 256, oLN = 320, oCK = 384, oCQ = 384 + kP64MaxCap,
                  oSC = 384 + 2 * kP64MaxCap, oRED = oSC + 4;

    constexpr int kEntryBytes = D * (int)(sizeof(IO) + sizeof(UL)) + DL * 4;  // one log entry
    extern __shared__ __align__(128) unsigned char smem[];
    const int NB = cfg.n_base, NS = cfg.n_slots;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + kP64BarrierBytes - 16);
    int *max_len_s = reinterpret_cast<int *>(smem + kP64BarrierBytes - 32);
    unsigned char *slots = smem + kP64BarrierBytes;
    unsigned char *base_ring = slots + (size_t)NS * kP64SlotBytes;
    unsigned char *aux_ring = base_ring + (size_t)NB * kChunkBytes;

    const uint32_t full_base = smem_addr(bars), empty_base = full_base + 8u * NB;
    const uint32_t full_key = empty_base + 8u * NB, empty_key = full_key + 8u * kP64MaxKey;
    const uint32_t full_val = empty_key + 8u * kP64MaxKey, empty_val = full_val + 8u * kP64MaxVal;
    const uint32_t prep_done = empty_val + 8u * kP64MaxVal;  // [NS] prep warp -> stream warp
    const uint32_t stream_done = prep_done + 8u * NS;   // [NS] stream warp -> epilogue warp
    const uint32_t coef_done = stream_done + 8u * NS;   // [NS] prep warp -> epilogue warp
    const uint32_t slot_free = coef_done + 8u * NS;     // [NS] epilogue warp -> prep warp

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) {
        for (int i = 0; i < NB; ++i) {
            mbar_init(full_base + 8u * i, 1);
            mbar_init(empty_base + 8u * i, 1);  // the unit's stream warp
        }
        for (int i = 0; i < kP64MaxKey; ++i) {
            mbar_init(full_key + 8u * i, 1);
            mbar_init(empty_key + 8u * i, 1);  // the unit's prep warp
        }
        for (int i = 0; i < kP64MaxVal; ++i) {
            mbar_init(full_val + 8u * i, 1);
            mbar_init(empty_val + 8u * i, 1);  // the unit's epilogue warp
        }
        for (int i = 0; i < NS; ++i) {
            mbar_init(prep_done + 8u * i, 1);
            mbar_init(stream_done + 8u * i, 1);
            mbar_init(coef_done + 8u * i, 1);
            mbar_init(slot_free + 8u * i, 1);
        }
        abort_flag[0] = 0;
        abort_flag[1] = 0;
        *max_len_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
    }
    __syncthreads();
    asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");  // see DELTALOG_HINT_BASE_UNTOUCHED

    const int total = tk.B * st.H;
    const bool slots_early = tk.slot_idx == nullptr || (tk.hints & DELTALOG_HINT_SLOTS_STABLE) != 0;
    // units blockIdx.x, blockIdx.x + gridDim.x, ... -- counted from the last unit downwards under DELTALOG_HINT_WALK_DOWN
    const int n_items = (int)blockIdx.x < total ? (total - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
    const bool walk_down = (tk.hints & DELTALOG_HINT_WALK_DOWN) != 0;
    const int first = walk_down ? total - 1 - (int)blockIdx.x : (int)blockIdx.x;
    const int stride = walk_down ? -(int)gridDim.x : (int)gridDim.x;
    const int cap = st.cap, H = st.H;
    auto slot_of = [&](int i) { return reinterpret_cast<float *>(slots + (size_t)(i % NS) * kP64SlotBytes); };
    constexpr int kFirstBaseWarp = kP64StreamWarps + 2 * kP64ScalarWarps;
    const bool is_base_producer = warp >= kFirstBaseWarp && warp < kFirstBaseWarp + kP64BaseWarps;

    // ---- prologue of every role but the base producers: the longest live log among this CTA's units -----
    // Lengths are written by the step before this one, so this is also where a kernel that was started
    // ahead of the preceding kernel's completion waits for it.  The aux producers look the lengths up (one
    // unit per lane), the maximum is combined in shared memory, and the aux ring is laid out for it.
    int NK = 4, NV = 4;  // depths of the key-side and the value-side ring
    int stage_cap = 1;   // entries a stage has room for
    if (!is_base_producer) {
        asm volatile("griddepcontrol.wait;\n" ::: "memory");
        if (warp >= kFirstBaseWarp + kP64BaseWarps) {
            const int a = warp - (kFirstBaseWarp + kP64BaseWarps);
            int mx = 0;
            for (int it = a * 32 + lane; it < n_items; it += 32 * kP64AuxWarps) {
                const int item = first + it * stride;
                const int slot = tk.slot_idx ? tk.slot_idx[item / H] : item / H;
                if (slot >= 0 && slot < st.num_slots) {
                    const int len = st.log_len[(size_t)slot * H + item % H];
                    if (len > 0 && len < cap) mx = max(mx, len);
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            if (lane == 0 && mx > 0) atomicMax(max_len_s, mx);
        }
        asm volatile("bar.sync 2, %0;\n" ::"n"(kP64Threads - 32 * kP64BaseWarps) : "memory");
        stage_cap = max(*max_len_s, 1);
        if (!kVecDecay) stage_cap = align_up(stage_cap, 4);  // scalar snapshots travel in 16-byte pieces
        if (stage_cap > cap) stage_cap = cap;
        // Depths (multiples of 4): a key-side stage is occupied for about 3 us (its copies' latency and the
        // prep warp), a value-side stage for about 5 us, so the unit rate is min(NK / 3, NV / 5) per
        // microsecond -- take the split that maximises it.  (Measured at 15 live entries of configuration 3:
        // depths 4 / 20 run at 101 us per launch, 8 / 8 at 75.)
        const int kb = KeyStage<OP, IO>(stage_cap).bytes, vb = ValStage<IO, UL>(stage_cap).bytes;
        int best = 0;
        for (int nk = 4; nk <= kP64MaxKey; nk += 4) {
            const int nv = min(kP64MaxVal, (cfg.aux_bytes - nk * kb) / vb) & ~3;
            if (nv < 4) break;
            const int rate = min(5 * nk, 3 * nv);
            if (rate > best) best = rate, NK = nk, NV = nv;
        }
    }
    const KeyStage<OP, IO> klay(stage_cap);
    const ValStage<IO, UL> vlay(stage_cap);
    unsigned char *key_ring = aux_ring;
    unsigned char *val_ring = aux_ring + (size_t)NK * klay.bytes;

    if (warp >= kP64StreamWarps + 2 * kP64ScalarWarps && warp < kP64StreamWarps + 2 * kP64ScalarWarps + kP64BaseWarps) {
        // ================= base producers: warp b owns units b, b + kP64BaseWarps, ... ==============
        // Unit i uses stage i % NB whether it is a padding row or not, so every role finds a unit's
        // stage from its index; one lane issues, so a warp never waits on itself whatever the ring depth.
        const int b = warp - (kP64StreamWarps + 2 * kP64ScalarWarps);
        bool dead = false;
        int n_q = 0;  // own units queued so far
        // tiles stream through L2 as first-to-evict (they are read once per launch), except for the fraction
        // the launcher asks L2 to hold on to across steps
        const float pin_fraction = fminf(1.f, st.l2_pin_bytes / ((float)total * (float)kChunkBytes));
        const uint64_t stream_policy = pin_fraction > 0.f ? l2_policy_keep(pin_fraction) : l2_policy_evict_first();
        if (!slots_early) asm volatile("griddepcontrol.wait;\n" ::: "memory");
        for (int n0 = 0; b + kP64BaseWarps * n0 < n_items; n0 += 32) {
            int slot = -1;
            const int my_it = b + kP64BaseWarps * (n0 + lane);
            if (my_it < n_items) {
                const int item = first + my_it * stride;
                slot = tk.slot_idx ? tk.slot_idx[item / H] : item / H;
                if (slot >= st.num_slots) slot = -1;
            }
            const int cnt = min(32, (n_items - b - kP64BaseWarps * n0 + kP64BaseWarps - 1) / kP64BaseWarps);
            for (int j = 0; j < cnt; ++j) {
                const int s = __shfl_sync(0xffffffffu, slot, j);
                if (lane != 0 || dead) continue;
                const int i = b + kP64BaseWarps * (n0 + j);
                const int stage = i % NB;
                if (!bounded_wait(empty_base + 8u * stage, ((uint32_t)(i / NB) & 1u) ^ 1u, abort_flag)) {
                    dead = true;
                    continue;
                }
                const uint32_t fb = full_base + 8u * stage;
                if (s < 0) {
                    mbar_arrive(fb);  // padding row: the stage passes empty
                } else {
                    const int h = (first + i * stride) % H;
                    mbar_arrive_expect_tx(fb, kChunkBytes);
                    bulk_copy_g2s_hint(smem_addr(base_ring + (size_t)stage * kChunkBytes),
                                       static_cast<const float *>(st.S_base) + ((size_t)s * H + h) * D * D, kChunkBytes, fb,
                                       stream_policy);
                }
                ++n_q;
            }
        }
        if (lane == 0 && dead) {
            if (st.status) atomicOr(st.status, DELTALOG_STATUS_TIMEOUT);
            // tiles this warp queued may still be in flight: wait (bounded) for those whose stage has not
            // been reused since (within NB units of the newest) to land
            for (int k = 0; k < n_q && kP64BaseWarps * k < NB; ++k) {
                const int i = b + kP64BaseWarps * (n_q - 1 - k);
                bounded_wait(full_base + 8u * (i % NB), (uint32_t)(i / NB) & 1u, abort_flag + 1);
            }
        }
    } else if (warp >= kP64StreamWarps + 2 * kP64ScalarWarps + kP64BaseWarps) {
        // ================= aux producers: warp a owns units a, a + kP64AuxWarps, ... ================
        const int a = warp - (kP64StreamWarps + 2 * kP64ScalarWarps + kP64BaseWarps);
        bool dead = false;
        const int io_vec = D * (int)sizeof(IO);
        int n_done = 0;
        for (int n0 = 0; a + kP64AuxWarps * n0 < n_items; n0 += 32) {
            int slot = -1, len = 0, flags = kMetaSkip, item = 0;
            float gs = 0.f, bt = 0.f;
            const int my_it = a + kP64AuxWarps * (n0 + lane);
            if (my_it < n_items) {
                item = first + my_it * stride;
                slot = tk.slot_idx ? tk.slot_idx[item / H] : item / H;
                if (slot >= st.num_slots) {
                    if (st.status) atomicOr(st.status, DELTALOG_STATUS_BAD_SLOT);
                    slot = -1;
                }
            }
            if (slot >= 0) {   // (the prologue has waited for the preceding kernel)
                if (!kVecDecay && tk.g) gs = tk.g[item];
                if (kDelta) bt = tk.beta[item];
                len = st.log_len[(size_t)slot * H + item % H];
                flags = 0;
                if (len >= cap || len < 0) {
                    if (st.status) atomicOr(st.status, DELTALOG_STATUS_LOG_FULL);
                    flags = kMetaFull;
                }
            }
            const int cnt = min(32, (n_items - a - kP64AuxWarps * n0 + kP64AuxWarps - 1) / kP64AuxWarps);
            for (int j = 0; j < cnt; ++j) {
                const int s = __shfl_sync(0xffffffffu, slot, j);
                const int L = __shfl_sync(0xffffffffu, len, j);
                const int fl = __shfl_sync(0xffffffffu, flags, j);
                const float gsj = __shfl_sync(0xffffffffu, gs, j);
                const float btj = __shfl_sync(0xffffffffu, bt, j);
                if (lane != 0 || dead) continue;
                const int i = a + kP64AuxWarps * (n0 + j);
                const int ks = i % NK, vs = i % NV;
                if (!bounded_wait(empty_key + 8u * ks, ((uint32_t)(i / NK) & 1u) ^ 1u, abort_flag) ||
                    !bounded_wait(empty_val + 8u * vs, ((uint32_t)(i / NV) & 1u) ^ 1u, abort_flag)) {
                    dead = true;
                    continue;
                }
                unsigned char *kst = key_ring + (size_t)ks * klay.bytes, *vst = val_ring + (size_t)vs * vlay.bytes;
                const uint32_t fk = full_key + 8u * ks, fv = full_val + 8u * vs;
                const int4 meta = make_int4(L, fl, __float_as_int(gsj), __float_as_int(btj));
                *reinterpret_cast<int4 *>(kst + klay.meta) = meta;
                *reinterpret_cast<int4 *>(vst + vlay.meta) = meta;
                *reinterpret_cast<int *>(vst + vlay.meta + 16) = s;
                if (fl != 0) {
                    mbar_arrive(fk);  // nothing to copy: the compute warps only read the flags
                    mbar_arrive(fv);
                } else {
                    const int item = first + i * stride;
                    const int kb = L * D * (int)sizeof(IO), ub = L * D * (int)sizeof(UL);
                    const int lb = kVecDecay ? L * D * 4 : align_up(L, 4) * 4;
                    mbar_arrive_expect_tx(fk, (L > 0 ? kb + lb : 0) + 2 * io_vec + (kVecDecay ? D * 4 : 0) +
                                                  (OP == DELTALOG_RWKV6 ? D * 4 : 0));
                    mbar_arrive_expect_tx(fv, (L > 0 ? ub : 0) + io_vec);
                    const size_t unit = (size_t)s * H + item % H;
                    const size_t qk = tk.qk_row(item / H, item % H);
                    const uint32_t ka = smem_addr(kst), va = smem_addr(vst);
                    bulk_copy_g2s(ka + klay.q, static_cast<const IO *>(tk.q) + qk * D, io_vec, fk);
                    bulk_copy_g2s(ka + klay.k, static_cast<const IO *>(tk.k) + qk * D, io_vec, fk);
                    if (kVecDecay) bulk_copy_g2s(ka + klay.g, tk.g + (size_t)item * D, D * 4, fk);
                    if (L > 0) {  // read again by the following steps: kept in L2 as far as it fits
                        const uint64_t keep = l2_policy_keep(st.keep_fraction(L, total, kEntryBytes));
                        bulk_copy_g2s_hint(ka + klay.L, st.decay_log + unit * cap * DL, lb, fk, keep);
                        bulk_copy_g2s_hint(ka + klay.K, static_cast<const IO *>(st.K_log) + unit * cap * D, kb, fk, keep);
                        bulk_copy_g2s_hint(va + vlay.U, static_cast<const UL *>(st.U_log) + unit * cap * D, ub, fv, keep);
                    }
                    if (OP == DELTALOG_RWKV6) bulk_copy_g2s(ka + klay.bonus, tk.u_bonus + (size_t)(item % H) * D, D * 4, fk);
                    bulk_copy_g2s(va + vlay.v, static_cast<const IO *>(tk.v) + (size_t)item * D, io_vec, fv);
                }
                ++n_done;
            }
        }
        if (dead && lane == 0) {
            if (st.status) atomicOr(st.status, DELTALOG_STATUS_TIMEOUT);
            for (int b = 0; b < n_done; ++b) {  // let this warp's copies in flight land: its newest units, one per stage
                const int i = a + kP64AuxWarps * (n_done - 1 - b);
                if (kP64AuxWarps * b < NK) bounded_wait(full_key + 8u * (i % NK), (uint32_t)(i / NK) & 1u, abort_flag + 1);
                if (kP64AuxWarps * b < NV) bounded_wait(full_val + 8u * (i % NV), (uint32_t)(i / NV) & 1u, abort_flag + 1);
                if (kP64AuxWarps * b >= NV) break;
            }
        }
    } else if (warp < kP64StreamWarps) {
        // ================= stream warps: warp w owns units w, w + 8, ... ============================
        // A lane holds four columns and the rows [32 rsub, 32 rsub + 32); the two lanes that share a
        // column group combine through a shuffle.  No cross-warp reduction: the unit is this warp's.
        const int c4 = lane & 15, rsub = lane >> 4;
        for (int i = warp; i < n_items; i += kP64StreamWarps) {
            const int sl = i % NS, bst = i % NB;
            if (!bounded_wait(prep_done + 8u * sl, (uint32_t)(i / NS) & 1u, abort_flag)) break;
            if (!bounded_wait(full_base + 8u * bst, (uint32_t)(i / NB) & 1u, abort_flag)) break;
            float *slot = slot_of(i);
            const int flags = __float_as_int(slot[oSC + 1]);
            if (flags == 0) {
                const float4 *tile = reinterpret_cast<const float4 *>(base_ring + (size_t)bst * kChunkBytes);
                float4 ak = make_float4(0.f, 0.f, 0.f, 0.f), aq = ak;
#pragma unroll 2
                for (int p4 = 0; p4 < 8; ++p4) {  // four consecutive rows at a time
                    const int r0 = 32 * rsub + 4 * p4;
                    const float4 mq4 = *reinterpret_cast<const float4 *>(slot + oMQ + r0);
                    float4 mk4 = mq4;
                    if (kDelta) mk4 = *reinterpret_cast<const float4 *>(slot + oMK + r0);
                    const float4 x0 = tile[(r0 + 0) * 16 + c4], x1 = tile[(r0 + 1) * 16 + c4];
                    const float4 x2 = tile[(r0 + 2) * 16 + c4], x3 = tile[(r0 + 3) * 16 + c4];
                    if (kDelta) {
                        ak = fma4(mk4.x, x0, ak);
                        ak = fma4(mk4.y, x1, ak);
                        ak = fma4(mk4.z, x2, ak);
                        ak = fma4(mk4.w, x3, ak);
                    }
                    aq = fma4(mq4.x, x0, aq);
                    aq = fma4(mq4.y, x1, aq);
                    aq = fma4(mq4.z, x2, aq);
                    aq = fma4(mq4.w, x3, aq);
                }
                if (kDelta) {
                    ak.x += __shfl_xor_sync(0xffffffffu, ak.x, 16);
                    ak.y += __shfl_xor_sync(0xffffffffu, ak.y, 16);
                    ak.z += __shfl_xor_sync(0xffffffffu, ak.z, 16);
                    ak.w += __shfl_xor_sync(0xffffffffu, ak.w, 16);
                }
                aq.x += __shfl_xor_sync(0xffffffffu, aq.x, 16);
                aq.y += __shfl_xor_sync(0xffffffffu, aq.y, 16);
                aq.z += __shfl_xor_sync(0xffffffffu, aq.z, 16);
                aq.w += __shfl_xor_sync(0xffffffffu, aq.w, 16);
                if (rsub == 0) {
                    float4 *red4 = reinterpret_cast<float4 *>(slot + oRED);
                    if (kDelta) red4[c4] = ak;
                    red4[16 + c4] = aq;
                }
            }
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(empty_base + 8u * bst);
                mbar_arrive(stream_done + 8u * sl);
            }
        }
    } else if (warp < kP64StreamWarps + kP64ScalarWarps) {
        // ================= prep warps: warp p owns units p, p + 4, ... =============================
        const int pw = warp - kP64StreamWarps;
        bool alive = true;
        for (int i = pw; i < n_items && alive; i += kP64ScalarWarps) {
            const int ks = i % NK, sl = i % NS;
            alive = bounded_wait(full_key + 8u * ks, (uint32_t)(i / NK) & 1u, abort_flag) &&
                    bounded_wait(slot_free + 8u * sl, ((uint32_t)(i / NS) & 1u) ^ 1u, abort_flag);
            if (!alive) break;
            const unsigned char *stage = key_ring + (size_t)ks * klay.bytes;
            const KeyStage<OP, IO> &lay = klay;
            float *slot = slot_of(i);
            const int4 meta = *reinterpret_cast<const int4 *>(stage + lay.meta);
            const int len = meta.x, flags = meta.y;
            if (flags == 0) {
                const IO *q_a = reinterpret_cast<const IO *>(stage + lay.q);
                const IO *k_a = reinterpret_cast<const IO *>(stage + lay.k);
                const IO *K_a = reinterpret_cast<const IO *>(stage + lay.K);
                const float *L_a = reinterpret_cast<const float *>(stage + lay.L);
                const float *g_a = reinterpret_cast<const float *>(stage + lay.g);
                const float *bonus_a = reinterpret_cast<const float *>(stage + lay.bonus);
                float qv[2], kv[2], lb[2];
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int jj = lane + 32 * e;
                    qv[e] = to_f32(q_a[jj]);
                    kv[e] = to_f32(k_a[jj]);
                    const float lold = (len > 0) ? L_a[(len - 1) * DL + (kVecDecay ? jj : 0)] : 0.f;
                    const float lnew = lold + (kVecDecay ? g_a[jj] : __int_as_float(meta.z));
                    lb[e] = kPost ? lnew : lold;  // the decay level the readouts refer to
                    const float ex = expf(lb[e]);
                    slot[oQ + jj] = qv[e];
                    slot[oK + jj] = kv[e];
                    slot[oLN + jj] = lnew;
                    slot[oLB + jj] = lb[e];
                    slot[oMK + jj] = ex * kv[e];
                    slot[oMQ + jj] = ex * qv[e];
                }
                if (lane == 0) slot[oSC + 1] = __int_as_float(0);
                __syncwarp();
                if (lane == 0) mbar_arrive(prep_done + 8u * sl);  // the stream group may start on this unit
                // Key-side replay coefficients, four entries per pass: eight lanes share an entry, a lane takes
                // eight consecutive key channels (one 16-byte load of the stored key, two of its snapshot), and
                // the sums are combined in three shuffle rounds.  (One entry per pass with a warp-wide
                // reduction cost ~280 cycles per entry, a dependent chain load -> exp -> five shuffle rounds,
                // and made this warp the slowest stage of the pipeline from eight live entries on.)
                {
                    const int s8 = lane & 7, e4 = lane >> 3;
                    float q8[8], k8[8], lb8[8];
                    load8(slot + oQ + 8 * s8, q8);
                    load8(slot + oK + 8 * s8, k8);
                    load8(slot + oLB + 8 * s8, lb8);
#pragma unroll 2
                    for (int i0 = 0; i0 < len; i0 += 4) {
                        const int i = i0 + e4;
                        float dq = 0.f, dk = 0.f;
                        if (i < len) {
                            float ke[8];
                            load8(K_a + i * D + 8 * s8, ke);
                            if (kVecDecay) {
                                float le[8];
                                load8(L_a + i * D + 8 * s8, le);
#pragma unroll
                                for (int e = 0; e < 8; ++e) ke[e] *= expf(lb8[e] - le[e]);
                            }
#pragma unroll
                            for (int e = 0; e < 8; ++e) {
                                dq = fmaf(q8[e], ke[e], dq);
                                if (kDelta) dk = fmaf(k8[e], ke[e], dk);
                            }
                        }
#pragma unroll
                        for (int o = 1; o < 8; o <<= 1) {
                            dq += __shfl_xor_sync(0xffffffffu, dq, o);
                            if (kDelta) dk += __shfl_xor_sync(0xffffffffu, dk, o);
                        }
                        if (s8 == 0 && i < len) {
                            const float w = kVecDecay ? 1.f : expf(lb8[0] - L_a[i]);
                            slot[oCQ + i] = w * dq;
                            if (kDelta) slot[oCK + i] = w * dk;
                        }
                    }
                }
                float d = 0.f;  // q.k for the readout from the updated state, r.(bonus.k) for RWKV6
#pragma unroll
                for (int e = 0; e < 2; ++e) d = fmaf(kPost ? qv[e] : qv[e] * bonus_a[lane + 32 * e], kv[e], d);
                d = warp_sum(d);
                if (lane == 0) slot[oSC] = d;
            } else if (lane == 0) {
                slot[oSC + 1] = __int_as_float(flags);
                mbar_arrive(prep_done + 8u * sl);
            }
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(coef_done + 8u * sl);
                mbar_arrive(empty_key + 8u * ks);   // the key side is not needed any more: its stage is free
            }
        }
        if (!alive && lane == 0 && st.status) atomicOr(st.status, DELTALOG_STATUS_TIMEOUT);
    } else {
        // ================= epilogue warps: warp e owns units e, e + 4, ... ==========================
        const int ew = warp - kP64StreamWarps - kP64ScalarWarps;
        bool alive = true;
        for (int i = ew; i < n_items && alive; i += kP64ScalarWarps) {
            const int vs = i % NV, sl = i % NS;
            const uint32_t par = (uint32_t)(i / NS) & 1u;
            alive = bounded_wait(stream_done + 8u * sl, par, abort_flag) &&
                    bounded_wait(coef_done + 8u * sl, par, abort_flag) &&
                    bounded_wait(full_val + 8u * vs, (uint32_t)(i / NV) & 1u, abort_flag);
            if (!alive) break;
            const unsigned char *stage = val_ring + (size_t)vs * vlay.bytes;
            const ValStage<IO, UL> &lay = vlay;
            const float *slot = slot_of(i);
            const int4 meta = *reinterpret_cast<const int4 *>(stage + lay.meta);
            const int len = meta.x, flags = meta.y;
            if (flags == 0) {
                const int slot_id = *reinterpret_cast<const int *>(stage + lay.meta + 16);
                const int item = first + i * stride;
                const size_t unit = (size_t)slot_id * H + item % H;
                const IO *v_a = reinterpret_cast<const IO *>(stage + lay.v);
                const UL *U_a = reinterpret_cast<const UL *>(stage + lay.U);
                const float *red_s = slot + oRED;
                UL *Uout = static_cast<UL *>(st.U_log) + (unit * cap + len) * D;
                IO *Kout = static_cast<IO *>(st.K_log) + (unit * cap + len) * D;
                IO *og = static_cast<IO *>(tk.out) + (size_t)item * D;
                // the new entry is read again by the following steps: same L2 policy as the log's reads
                const uint64_t keep = l2_policy_keep(st.keep_fraction(len + 1, total, kEntryBytes));
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int c = lane + 32 * e;  // this lane's output column
                    float yk = kDelta ? red_s[c] : 0.f, yq = red_s[D + c];
                    for (int e0 = 0; e0 < len; ++e0) {
                        const float u = to_f32(U_a[e0 * D + c]);
                        if (kDelta) yk = fmaf(slot[oCK + e0], u, yk);
                        yq = fmaf(slot[oCQ + e0], u, yq);
                    }
                    const IO v_raw = v_a[c];
                    if (kDelta) {
                        const float bval = __int_as_float(meta.w) * (to_f32(v_raw) - yk);
                        st_hint(Uout + c, from_f32<UL>(bval), keep);
                        og[c] = from_f32<IO>(st.scale * fmaf(slot[oSC], bval, yq));
                    } else {
                        st_hint(Uout + c, from_f32<UL>(to_f32(v_raw)), keep);  // lossless: U log dtype equals the I/O dtype
                        og[c] = from_f32<IO>((kPost ? st.scale : 1.f) * fmaf(slot[oSC], to_f32(v_raw), yq));
                    }
                    st_hint(Kout + c, from_f32<IO>(slot[oK + c]), keep);  // the key as the prep warp widened it: exact
                    if (kVecDecay) st_hint(st.decay_log + (unit * cap + len) * DL + c, slot[oLN + c], keep);
                }
                if (lane == 0) {
                    if (!kVecDecay) st_hint(st.decay_log + unit * cap + len, slot[oLN], keep);
                    st.log_len[unit] = len + 1;
                }
            }
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(slot_free + 8u * sl);
                mbar_arrive(empty_val + 8u * vs);
            }
        }
        if (!alive && lane == 0 && st.status) atomicOr(st.status, DELTALOG_STATUS_TIMEOUT);
    }
}

}  // namespace deltalog
