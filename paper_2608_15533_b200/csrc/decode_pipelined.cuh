// Persistent, warp-specialised decode + append kernel (head size 128).
//
// Same arithmetic as decode_append_kernel (Algorithm 1, append branch; Eq. 4 and Eq. 6), different
// schedule.  One CTA stays resident per SM and walks over its share of the (batch row, head) units.
// Five roles run concurrently and hand work to one another through mbarriers:
//
//   base producers (4 warps) bulk asynchronous copies (cp.async.bulk, completion counted on
//                            mbarriers) of 16 KiB chunks of the base tile (fp32: four chunks, bf16:
//                            two) -- the only large read -- into the base ring, warp c bringing
//                            chunk c of every unit; a
//                            chunk's stage is refilled the moment that chunk has been consumed, so
//                            the HBM stream never waits for a unit's epilogue or for a whole tile;
//   aux producers  (2 warps) per unit: the live log entries K[0:len], U[0:len], Lambda[0:len], the
//                            token vectors q, k, v (and g, bonus where they are vectors) and a small
//                            metadata record written by the producer (len, flags, scalar gate, beta)
//                            into the aux ring; the warps take the units in turn (a trace showed one
//                            thread needing 1 - 1.5 us for a unit's seven copies beside the busy
//                            compute warps: enough for an fp32 base tile, not for a bf16 one);
//   stream group   (8 warps) the base pass only: the two mat-vecs S_base^T (e^lbar . k) and
//                            S_base^T (e^lbar . q) from each chunk as it lands;
//   prep group     (4 warps) for unit i+1: cumulative decay, decayed multipliers (handed to the
//                            stream group) and the key-side replay coefficients -- the paper's
//                            ReplayPrep, here a pipeline stage instead of a launch;
//   epilogue group (4 warps) for unit i, once the stream group is through it: cross-warp
//                            reduction, value-side replay, b, the output and the append.
//
// No compute warp ever issues a global load; what the epilogue group writes (out, the appended
// entry and the new length) is fire-and-forget.  Every wait on an mbarrier is bounded in time:
// when it gives up it raises the CTA's abort flag, ORs DELTALOG_STATUS_TIMEOUT into the status
// word, and all roles leave their loops.
#pragma once

#include "common.cuh"

namespace deltalog {

constexpr int kChunkBytes = 16384;
// Bytes of one base-ring stage: a whole number of tile rows, at most kChunkBytes.
template <int D, typename BT>
__host__ __device__ constexpr int chunk_bytes() {
    return D * D * (int)sizeof(BT) < kChunkBytes ? D * D * (int)sizeof(BT) : kChunkBytes;
}
constexpr int kPipeConsumers = 256;                    // threads of the stream group and of the scalar group
constexpr int kBaseWarps = 4;                          // base-ring producer warps: one per chunk of a tile
#ifndef DELTALOG_AUX_WARPS
#define DELTALOG_AUX_WARPS 2
#endif
constexpr int kAuxWarps = DELTALOG_AUX_WARPS;          // aux-ring producer warps: they take the units in turn
constexpr int kPipeThreads = 2 * kPipeConsumers + 32 * (kBaseWarps + kAuxWarps);  // + base and aux producers
// Upper bound on any single wait inside the kernel (compile-time knob; the give-up path is exercised by a
// test build with a limit of a few milliseconds).
#ifndef DELTALOG_WAIT_LIMIT_NS
#define DELTALOG_WAIT_LIMIT_NS 2000000000ull  // 2 s per wait
#endif
constexpr unsigned long long kWaitLimitNs = DELTALOG_WAIT_LIMIT_NS;
// Test builds only (-DDELTALOG_TEST_HOOKS=1): PipeCfg.test_drop_item names one unit (global index) whose
// chunk 0 the base producer never requests, so that the stream group's wait for it runs out -- the only
// way to see the give-up path of the bounded waits without hanging or faulting anything.
#ifndef DELTALOG_TEST_HOOKS
#define DELTALOG_TEST_HOOKS 0
#endif

enum : int { kMetaSkip = 1, kMetaFull = 2 };

__host__ __device__ constexpr int align_up(int x, int a) { return (x + a - 1) / a * a; }

// Byte offsets inside one aux-ring stage (all multiples of 16).
template <int OP, int D, typename IO, typename UL>
struct AuxLayout {
    static constexpr bool kVec = OpTraits<OP>::kVecDecay;
    static constexpr int DL = kVec ? D : 1;
    int K, U, L, q, k, v, g, bonus, meta, bytes;
    __host__ __device__ explicit AuxLayout(int cap) {
        K = 0;
        U = K + cap * D * (int)sizeof(IO);
        L = U + cap * D * (int)sizeof(UL);
        q = L + align_up(cap * DL * 4, 16);
        k = q + D * (int)sizeof(IO);
        v = k + D * (int)sizeof(IO);
        g = v + D * (int)sizeof(IO);
        bonus = g + (kVec ? D * 4 : 0);
        meta = bonus + (OP == DELTALOG_RWKV6 ? D * 4 : 0);
        bytes = align_up(meta + 32, 128);
    }
};

// Hand-over buffer between the roles: 1 << slot_shift slots (as many units are in flight between
// the prep group and the epilogue group; two suffice while a unit's base tile takes longer to
// arrive than the chain prep -> stream -> epilogue takes, four are used with a 16-bit base).
// Per slot (floats): q, k, mul_k, mul_q, lbar, lbar' [6*D], ck, cq [2*64], scalars [4]: q.k and the
// unit's flags; then the stream group's partial sums [RL][2][D].
template <int D>
__host__ __device__ constexpr int pipe_slot_floats() {
    return 6 * D + 2 * kMaxCap + 4 + 2 * D * (kPipeConsumers / (D / 4));
}
template <int D>
__host__ __device__ constexpr int pipe_scratch_bytes(int slot_shift) {
    return (1 << slot_shift) * align_up(pipe_slot_floats<D>() * 4, 128);
}
constexpr int kPipeMaxBase = 32;         // upper bounds on the ring depths (mbarrier storage)
constexpr int kPipeMaxAux = 12;
constexpr int kPipeBarrierBytes = 1024;  // mbarriers (2 x 32 + 2 x 12 + 4 x 4 at most), the abort flags, the live-length word

struct PipeCfg {
    int n_base;     // stages of the base ring
    int aux_bytes;  // bytes of the aux ring's region; its depth follows from the live log lengths (see the kernel)
    int slot_shift;  // log2 of the number of hand-over slots (1 or 2)
    int test_drop_item;  // -1; a unit index only in test builds (DELTALOG_TEST_HOOKS)
};

template <int D, typename BT = float>
__host__ inline int pipe_smem_bytes(PipeCfg cfg) {
    return kPipeBarrierBytes + pipe_scratch_bytes<D>(cfg.slot_shift) + cfg.n_base * chunk_bytes<D, BT>() + cfg.aux_bytes;
}

// ---- mbarrier / bulk-copy primitives ---------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bulk asynchronous copy global -> this CTA's shared memory; bytes % 16 == 0, both addresses 16-byte aligned.
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
// The same with an L2 eviction policy for the lines the copy brings in.
__device__ __forceinline__ void bulk_copy_g2s_hint(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar,
                                                   uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;\n" ::"r"(dst),
        "l"(src), "r"(bytes), "r"(bar), "l"(policy)
        : "memory");
}
__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;\n" : "=l"(t));
    return t;
}

// Wait for a phase of an mbarrier, giving up after kWaitLimitNs or as soon as the CTA aborts.
// (The polling loop is kept out of line: the kernel's roles share the SM's instruction caches, and a
// dozen inlined copies of it were a measurable part of the instruction-fetch traffic.)
static __device__ __noinline__ bool bounded_wait_slow(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
    const unsigned long long t0 = global_timer_ns();
    for (uint32_t spin = 1;; ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((spin & 63u) == 0) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > kWaitLimitNs) {
                *abort_flag = 1;
                return false;
            }
        }
    }
}
__device__ __forceinline__ bool bounded_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    return bounded_wait_slow(bar, parity, abort_flag);
}

// OR-reduction of a predicate over the consumer warps (named barrier 1), also a consumer-only barrier.
__device__ __forceinline__ bool consumers_any(bool pred) {
    uint32_t res;
    asm volatile(
        "{\n .reg .pred p, q;\n setp.ne.u32 q, %1, 0;\n bar.red.or.pred p, 1, %2, q;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(res)
        : "r"((uint32_t)pred), "n"(kPipeConsumers)
        : "memory");
    return res != 0;
}
__device__ __forceinline__ void consumers_sync() {
    asm volatile("bar.sync 1, %0;\n" ::"n"(kPipeConsumers) : "memory");
}

// The same for one of the two 128-thread scalar groups (named barrier `id`).
__device__ __forceinline__ bool group_any(bool pred, int id) {
    uint32_t res;
    asm volatile(
        "{\n .reg .pred p, q;\n setp.ne.u32 q, %1, 0;\n bar.red.or.pred p, %2, 128, q;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(res)
        : "r"((uint32_t)pred), "r"(id)
        : "memory");
    return res != 0;
}
__device__ __forceinline__ void group_sync(int id) { asm volatile("bar.sync %0, 128;\n" ::"r"(id) : "memory"); }

struct RingPos {  // position in a ring of n stages: stage index and phase parity
    int stage = 0;
    uint32_t phase = 0;
    __device__ __forceinline__ void advance(int n) {
        if (++stage == n) {
            stage = 0;
            phase ^= 1u;
        }
    }
};

template <int OP, int D, typename IO, typename UL, typename BT = float>
__global__ void __launch_bounds__(kPipeThreads, 1)
decode_pipelined_kernel(StateArgs st, TokenArgs tk, PipeCfg cfg) {
    constexpr bool kDelta = OpTraits<OP>::kDeltaRule;
    constexpr bool kPost = OpTraits<OP>::kPostReadout;
    constexpr bool kVecDecay = OpTraits<OP>::kVecDecay;
    constexpr int DL = kVecDecay ? D : 1;
    constexpr int C4 = D / 4;
    constexpr int RL = kPipeConsumers / C4;          // row groups of the stream group
    constexpr int CHB = chunk_bytes<D, BT>();        // bytes per base-ring stage
    constexpr int NCHUNK = D * D * (int)sizeof(BT) / CHB;  // chunks per base tile
    constexpr int CH_ROWS = D / NCHUNK;              // rows per chunk
    constexpr int PPC = CH_ROWS / RL;                // rows of a chunk per stream thread
    static_assert(PPC % 4 == 0 && PPC * RL * NCHUNK == D, "the base pass takes a thread's rows four at a time");
    constexpr int EPL = D / 32;                      // key channels per lane in the coefficient phase
    constexpr int kEntryBytes = D * (int)(sizeof(IO) + sizeof(UL)) + DL * 4;  // one log entry
    constexpr int kGroupWarps = kPipeConsumers / 32;
    constexpr int SLOT = align_up(pipe_slot_floats<D>() * 4, 128) / 4;  // floats per hand-over slot

    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + kPipeBarrierBytes - 16);
    int *max_len_s = reinterpret_cast<int *>(smem + kPipeBarrierBytes - 32);
    float *scratch = reinterpret_cast<float *>(smem + kPipeBarrierBytes);
    unsigned char *base_ring = smem + kPipeBarrierBytes + pipe_scratch_bytes<D>(cfg.slot_shift);
    unsigned char *aux_ring = base_ring + (size_t)cfg.n_base * CHB;

    const int NB = cfg.n_base;
    const uint32_t full_base = smem_addr(bars), empty_base = full_base + 8u * NB;
    const uint32_t full_aux = empty_base + 8u * NB, empty_aux = full_aux + 8u * kPipeMaxAux;
    const int SH = cfg.slot_shift, NS = 1 << SH;      // hand-over slots; unit i uses slot i % NS in phase (i / NS) & 1
    const uint32_t prep_done = empty_aux + 8u * kPipeMaxAux;   // [NS] scalar group -> stream group: multipliers ready
    const uint32_t stream_done = prep_done + 8u * NS;  // [NS] stream group -> epilogue group: partial sums ready
    const uint32_t coef_done = stream_done + 8u * NS;  // [NS] prep group -> epilogue group: coefficients ready
    const uint32_t slot_free = coef_done + 8u * NS;    // [NS] epilogue group -> prep group: hand-over slot reusable

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) {
        for (int i = 0; i < NB; ++i) {
            mbar_init(full_base + 8u * i, 1);
            mbar_init(empty_base + 8u * i, kGroupWarps);
        }
        for (int i = 0; i < kPipeMaxAux; ++i) {
            mbar_init(full_aux + 8u * i, 1);
            mbar_init(empty_aux + 8u * i, kGroupWarps);
        }
        for (int i = 0; i < NS; ++i) {
            mbar_init(prep_done + 8u * i, 1);
            mbar_init(stream_done + 8u * i, kGroupWarps);
            mbar_init(coef_done + 8u * i, kGroupWarps / 2);
            mbar_init(slot_free + 8u * i, kGroupWarps / 2);
        }
        abort_flag[0] = 0;
        abort_flag[1] = 0;  // separate flag for the drain waits after an abort
        *max_len_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
    }
    __syncthreads();
    // Programmatic dependent launch: a kernel queued behind this one may start its CTAs as this one's
    // retire (it synchronises with griddepcontrol.wait before it touches anything written here).
    asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");

    const int total = tk.B * st.H;
    const bool slots_early = tk.slot_idx == nullptr || (tk.hints & DELTALOG_HINT_SLOTS_STABLE) != 0;
    // A CTA takes the units blockIdx.x, blockIdx.x + gridDim.x, ... -- counted from the last unit downwards under
    // DELTALOG_HINT_WALK_DOWN (unit = first + i * stride either way).
    const int n_items = (total - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    const bool walk_down = (tk.hints & DELTALOG_HINT_WALK_DOWN) != 0;
    const int first = walk_down ? total - 1 - (int)blockIdx.x : (int)blockIdx.x;
    const int stride = walk_down ? -(int)gridDim.x : (int)gridDim.x;
    const int cap = st.cap, H = st.H;

    // ---- the aux ring is laid out for the longest LIVE log among this CTA's units ----------------------
    // A unit's aux stage holds its live log entries and token vectors from the moment the copies are queued
    // until its epilogue is done; stages sized for the full capacity leave room for few of them at large
    // capacities (and used to shrink the base ring).  So the aux producers first look up the lengths of the
    // CTA's units -- which is also where a kernel started ahead of the preceding kernel's completion waits
    // for it: the lengths are written by the step before -- and every role but the base producers (the base
    // ring has a fixed place; its producers start at once) picks the depth up from shared memory.
    constexpr int kFirstBaseWarp = 2 * kGroupWarps, kFirstAuxWarp = 2 * kGroupWarps + kBaseWarps;
    const bool is_base_producer = warp >= kFirstBaseWarp && warp < kFirstAuxWarp;
    int NA = 2, stage_cap = 1;
    if (!is_base_producer) {
        if (warp >= kFirstAuxWarp) {
            asm volatile("griddepcontrol.wait;\n" ::: "memory");
            int mx = 0;
            for (int it = (warp - kFirstAuxWarp) * 32 + lane; it < n_items; it += 32 * kAuxWarps) {
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
        asm volatile("bar.sync 3, %0;\n" ::"n"(kPipeThreads - 32 * kBaseWarps) : "memory");
        stage_cap = max(*max_len_s, 1);
        if (!kVecDecay) stage_cap = align_up(stage_cap, 4);  // scalar snapshots travel in 16-byte pieces
        if (stage_cap > cap) stage_cap = cap;
        NA = min(kPipeMaxAux, cfg.aux_bytes / AuxLayout<OP, D, IO, UL>(stage_cap).bytes);  // >= 2: the launcher's check
    }
    const AuxLayout<OP, D, IO, UL> lay(stage_cap);

    // hand-over slot fields
    auto slot_ptr = [&](int i) { return scratch + (size_t)(i & (NS - 1)) * SLOT; };
    constexpr int oQ = 0, oK = D, oMK = 2 * D, oMQ = 3 * D, oLB = 4 * D, oLN = 5 * D, oCK = 6 * D,
                  oCQ = 6 * D + kMaxCap, oSC = 6 * D + 2 * kMaxCap, oRED = 6 * D + 2 * kMaxCap + 4;

    if (warp >= 2 * kGroupWarps && warp < 2 * kGroupWarps + kBaseWarps) {
        // ================= base-ring producers: need only the slot of each unit ===================
        // Warp c brings chunk c of every unit, on its own: a stage is refilled the moment the stream
        // group has released THAT chunk, not when the whole tile two units back has been consumed
        // (a trace showed the ring running two tiles deep at tile granularity: issue -> first chunk
        // 1.6 us, the stream group idle in between).  One lane per warp issues; a wait + arm + copy
        // costs it ~350 ns, one chunk per unit and warp is well inside the budget.
        static_assert(NCHUNK <= kBaseWarps, "one producer warp per chunk of a tile");
        const int c = warp - 2 * kGroupWarps;
        bool dead = false;
        int m = 0;  // units queued so far (warp-uniform)
        // every tile is read once per launch: first to be evicted from L2, so that the live log entries and
        // the length words, which the next step reads again, stay there
        // ... except for a fixed fraction of them (chosen by the hardware from the address), which is asked to
        // stay: what L2 can hold beside the log need not be fetched from HBM again by the next step
        const float pin_fraction = fminf(1.f, st.l2_pin_bytes / ((float)total * (float)(D * D) * (float)sizeof(BT)));
        const uint64_t stream_policy = pin_fraction > 0.f ? l2_policy_keep(pin_fraction) : l2_policy_evict_first();
        // Started ahead of the preceding kernel's completion (chained launch), these warps read two things
        // early: the slot list and the base tiles.  The caller vouched for the tiles
        // (DELTALOG_HINT_BASE_UNTOUCHED); the slot list may be read early only if there is none or the
        // caller vouched for it as well (DELTALOG_HINT_SLOTS_STABLE) -- otherwise wait here.
        if (!slots_early) asm volatile("griddepcontrol.wait;\n" ::: "memory");
        for (int it0 = 0; it0 < n_items && c < NCHUNK; it0 += 32) {
            int slot = -1;
            if (it0 + lane < n_items) {
                const int item = first + (it0 + lane) * stride;
                slot = tk.slot_idx ? tk.slot_idx[item / H] : item / H;
                if (slot >= st.num_slots) slot = -1;
            }
            const int cnt = min(32, n_items - it0);
            for (int j = 0; j < cnt; ++j) {
                const int s = __shfl_sync(0xffffffffu, slot, j);
                if (s < 0) continue;
#if DELTALOG_TEST_HOOKS
                if (c == 0 && first + (it0 + j) * stride == cfg.test_drop_item) dead = true;  // never requested
#endif
                if (lane == 0 && !dead) {
                    const int h = (first + (it0 + j) * stride) % H;
                    const char *src = static_cast<const char *>(st.S_base) + ((size_t)s * H + h) * D * D * sizeof(BT);
                    const int mm = m * NCHUNK + c;
                    const int stage = mm % NB;
                    const uint32_t phase = (uint32_t)(mm / NB) & 1u;
                    if (!bounded_wait(empty_base + 8u * stage, phase ^ 1u, abort_flag)) {
                        dead = true;
                    } else {
                        const uint32_t fb = full_base + 8u * stage;
                        mbar_arrive_expect_tx(fb, CHB);
#if DELTALOG_STREAM_BASE
                        bulk_copy_g2s_hint(smem_addr(base_ring + (size_t)stage * CHB), src + (size_t)c * CHB, CHB, fb, stream_policy);
#else
                        bulk_copy_g2s(smem_addr(base_ring + (size_t)stage * CHB), src + (size_t)c * CHB, CHB, fb);
#endif
                    }
                }
                if (!dead) ++m;  // lane 0: units whose chunk was queued
            }
        }
        if (lane == 0 && dead) {
            if (st.status) atomicOr(st.status, DELTALOG_STATUS_TIMEOUT);
            // chunks this warp queued may still be in flight: wait (bounded) for those whose stage has not
            // been reused since (within NB chunk indices of the newest) to land before the CTA may exit
            for (int i = 0; i < m && NCHUNK * i < NB; ++i) {
                const int mm = (m - 1 - i) * NCHUNK + c;
                bounded_wait(full_base + 8u * (mm % NB), (uint32_t)(mm / NB) & 1u, abort_flag + 1);
            }
        }
    } else if (warp >= 2 * kGroupWarps + kBaseWarps) {
        // ================= aux-ring producers: metadata, live log entries, token vectors =========
        // Warp a takes the units a, a + kAuxWarps, ... of this CTA; a unit's stage and phase follow from
        // its index alone, so the warps need not talk to one another.  (The one-bit phase parity of the
        // wait below stays unambiguous although a stage is awaited by different warps in turn: units are
        // consumed strictly in order, and before warp a waits for unit i's stage it has queued unit
        // i - kAuxWarps, so every unit up to i - kAuxWarps - NA -- which includes the user of this stage
        // before the previous one -- has been consumed: the waiter is never two phases off.)
        const int a = warp - (2 * kGroupWarps + kBaseWarps);
        bool dead = false;
        int n_done = 0;  // own units queued so far
        const int io_vec = D * (int)sizeof(IO);
        // Lengths and log entries are written by the step before this one, and the token tensors
        // (gate, beta, q, k, v) are typically produced by the launch directly in front of this one: these
        // warps have waited for the preceding kernel (in the prologue above) before any of them is read.
        // Everything the other roles do with global memory follows from what these warps load.
        for (int n0 = 0; a + kAuxWarps * n0 < n_items; n0 += 32) {
            int slot = -1, len = 0, flags = kMetaSkip, item = 0;
            float gs = 0.f, bt = 0.f;
            const int my_it = a + kAuxWarps * (n0 + lane);
            if (my_it < n_items) {
                item = first + my_it * stride;
                slot = tk.slot_idx ? tk.slot_idx[item / H] : item / H;
                if (slot >= st.num_slots) {
                    if (st.status) atomicOr(st.status, DELTALOG_STATUS_BAD_SLOT);
                    slot = -1;
                }
            }
            if (slot >= 0) {   // (these warps have waited for the preceding kernel in the prologue)
                if (!kVecDecay && tk.g) gs = tk.g[item];  // no gate: plain linear attention
                if (kDelta) bt = tk.beta[item];
                len = st.log_len[(size_t)slot * H + item % H];
                flags = 0;
                if (len >= cap || len < 0) {
                    if (st.status) atomicOr(st.status, DELTALOG_STATUS_LOG_FULL);
                    flags = kMetaFull;
                }
            }
            const int cnt = min(32, (n_items - a - kAuxWarps * n0 + kAuxWarps - 1) / kAuxWarps);
            for (int j = 0; j < cnt; ++j) {
                const int s = __shfl_sync(0xffffffffu, slot, j);
                const int L = __shfl_sync(0xffffffffu, len, j);
                const int fl = __shfl_sync(0xffffffffu, flags, j);
                const float gsj = __shfl_sync(0xffffffffu, gs, j);
                const float btj = __shfl_sync(0xffffffffu, bt, j);
                if (lane != 0 || dead) continue;
                const int it = a + kAuxWarps * (n0 + j);
                const int stg = it % NA;
                const uint32_t phase = (uint32_t)(it / NA) & 1u;
                if (!bounded_wait(empty_aux + 8u * stg, phase ^ 1u, abort_flag)) {
                    dead = true;
                    continue;
                }
                unsigned char *stage = aux_ring + (size_t)stg * lay.bytes;
                *reinterpret_cast<int4 *>(stage + lay.meta) = make_int4(L, fl, __float_as_int(gsj), __float_as_int(btj));
                *reinterpret_cast<int *>(stage + lay.meta + 16) = s;
                const uint32_t fa = full_aux + 8u * stg;
                if (fl != 0) {
                    mbar_arrive(fa);  // nothing to copy: the compute warps only read the flags
                } else {
                    const int item = first + it * stride;
                    const size_t unit = (size_t)s * H + item % H;
                    const int kb = L * D * (int)sizeof(IO), ub = L * D * (int)sizeof(UL);
                    const int lb = kVecDecay ? L * D * 4 : align_up(L, 4) * 4;
                    const uint32_t bytes = kb + ub + lb + 3 * io_vec + (kVecDecay ? D * 4 : 0) +
                                           (OP == DELTALOG_RWKV6 ? D * 4 : 0);
                    mbar_arrive_expect_tx(fa, bytes);
                    const uint32_t sa = smem_addr(stage);
                    const size_t qk = tk.qk_row(item / H, item % H);
                    bulk_copy_g2s(sa + lay.q, static_cast<const IO *>(tk.q) + qk * D, io_vec, fa);
                    bulk_copy_g2s(sa + lay.k, static_cast<const IO *>(tk.k) + qk * D, io_vec, fa);
                    if (kVecDecay) bulk_copy_g2s(sa + lay.g, tk.g + (size_t)item * D, D * 4, fa);
                    if (L > 0) {
#if DELTALOG_L2_KEEP
                        const uint64_t keep = l2_policy_keep(st.keep_fraction(L, total, kEntryBytes));
                        bulk_copy_g2s_hint(sa + lay.L, st.decay_log + unit * cap * DL, lb, fa, keep);
                        bulk_copy_g2s_hint(sa + lay.K, static_cast<const IO *>(st.K_log) + unit * cap * D, kb, fa, keep);
                        bulk_copy_g2s_hint(sa + lay.U, static_cast<const UL *>(st.U_log) + unit * cap * D, ub, fa, keep);
#else
                        bulk_copy_g2s(sa + lay.L, st.decay_log + unit * cap * DL, lb, fa);
                        bulk_copy_g2s(sa + lay.K, static_cast<const IO *>(st.K_log) + unit * cap * D, kb, fa);
                        bulk_copy_g2s(sa + lay.U, static_cast<const UL *>(st.U_log) + unit * cap * D, ub, fa);
#endif
                    }
                    bulk_copy_g2s(sa + lay.v, static_cast<const IO *>(tk.v) + (size_t)item * D, io_vec, fa);
                    if (OP == DELTALOG_RWKV6) bulk_copy_g2s(sa + lay.bonus, tk.u_bonus + (size_t)(item % H) * D, D * 4, fa);
                }
                ++n_done;
            }
        }
        if (lane == 0 && dead) {
            // wait (bounded) for this warp's copies still in flight: its last own units, at most one per stage
            if (st.status) atomicOr(st.status, DELTALOG_STATUS_TIMEOUT);
            for (int i = 0; i < n_done && kAuxWarps * i < NA; ++i) {  // units within NA of the newest: distinct stages
                const int it = a + kAuxWarps * (n_done - 1 - i);
                bounded_wait(full_aux + 8u * (it % NA), (uint32_t)(it / NA) & 1u, abort_flag + 1);
            }
        }
    } else if (warp < kGroupWarps) {
        // ================= stream group: the base pass, nothing else =============================
        // Warps run independently of one another (no group barrier): each waits for the unit's
        // multipliers, folds its rows of every chunk into its partial sums and hands them over.
        const int c4 = tid % C4, rl = tid / C4;
        RingPos bpos;
        for (int it = 0; it < n_items; ++it) {
            const uint32_t par = (uint32_t)(it >> SH) & 1u;
            if (!bounded_wait(prep_done + 8u * (it & (NS - 1)), par, abort_flag)) break;
            float *sl = slot_ptr(it);
            const int flags = __float_as_int(sl[oSC + 1]);
            if (!(flags & kMetaSkip)) {
                const float *mk_s = sl + oMK, *mq_s = sl + oMQ;
                float4 ak = make_float4(0.f, 0.f, 0.f, 0.f), aq = ak;
                // bf16 base: two rows per packed FMA (even-row and odd-row partial sums per column)
                float2 ak2[4], aq2[4];
#pragma unroll
                for (int x = 0; x < 4; ++x) ak2[x] = aq2[x] = make_float2(0.f, 0.f);
                bool failed = false;
#pragma unroll 1
                for (int c = 0; c < NCHUNK; ++c) {
                    if (!bounded_wait(full_base + 8u * bpos.stage, bpos.phase, abort_flag)) {
                        failed = true;
                        break;
                    }
                    if (!(flags & kMetaFull)) {
                        const BT *tile = reinterpret_cast<const BT *>(base_ring + (size_t)bpos.stage * CHB);
                        if constexpr (sizeof(BT) == 2) {
                            // With half the bytes per unit the instruction count starts to matter: rows are
                            // taken in pairs, the pair's multipliers come from shared memory as one float2 and
                            // one packed fp32 FMA serves both rows of a column.
#pragma unroll
                            for (int pg = 0; pg < PPC; pg += 2) {
                                const int rc = rl * PPC + pg, r0 = c * CH_ROWS + rc;
                                const float2 mq2 = *reinterpret_cast<const float2 *>(mq_s + r0);
                                float2 mk2 = mq2;
                                if (kDelta) mk2 = *reinterpret_cast<const float2 *>(mk_s + r0);
                                const uint2 a = *reinterpret_cast<const uint2 *>(tile + ((rc + 0) * C4 + c4) * 4);
                                const uint2 b = *reinterpret_cast<const uint2 *>(tile + ((rc + 1) * C4 + c4) * 4);
                                const float2 x0 = make_float2(__uint_as_float(a.x << 16), __uint_as_float(b.x << 16));
                                const float2 x1 = make_float2(__uint_as_float(a.x & 0xffff0000u), __uint_as_float(b.x & 0xffff0000u));
                                const float2 x2 = make_float2(__uint_as_float(a.y << 16), __uint_as_float(b.y << 16));
                                const float2 x3 = make_float2(__uint_as_float(a.y & 0xffff0000u), __uint_as_float(b.y & 0xffff0000u));
                                if (kDelta) {
                                    ak2[0] = __ffma2_rn(mk2, x0, ak2[0]);
                                    ak2[1] = __ffma2_rn(mk2, x1, ak2[1]);
                                    ak2[2] = __ffma2_rn(mk2, x2, ak2[2]);
                                    ak2[3] = __ffma2_rn(mk2, x3, ak2[3]);
                                }
                                aq2[0] = __ffma2_rn(mq2, x0, aq2[0]);
                                aq2[1] = __ffma2_rn(mq2, x1, aq2[1]);
                                aq2[2] = __ffma2_rn(mq2, x2, aq2[2]);
                                aq2[3] = __ffma2_rn(mq2, x3, aq2[3]);
                            }
                        } else {
#pragma unroll
                        for (int pg = 0; pg < PPC; pg += 4) {  // this thread's consecutive rows, four at a time
                            const int rc = rl * PPC + pg, r0 = c * CH_ROWS + rc;
                            const float4 mq4 = *reinterpret_cast<const float4 *>(mq_s + r0);
                            float4 mk4 = mq4;
                            if (kDelta) mk4 = *reinterpret_cast<const float4 *>(mk_s + r0);
                            const float4 x0 = base_load4<BT>(tile + ((rc + 0) * C4 + c4) * 4);
                            const float4 x1 = base_load4<BT>(tile + ((rc + 1) * C4 + c4) * 4);
                            const float4 x2 = base_load4<BT>(tile + ((rc + 2) * C4 + c4) * 4);
                            const float4 x3 = base_load4<BT>(tile + ((rc + 3) * C4 + c4) * 4);
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
                        }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(empty_base + 8u * bpos.stage);
                    bpos.advance(NB);
                }
                if (failed) break;
                if constexpr (sizeof(BT) == 2) {
                    ak = make_float4(ak2[0].x + ak2[0].y, ak2[1].x + ak2[1].y, ak2[2].x + ak2[2].y, ak2[3].x + ak2[3].y);
                    aq = make_float4(aq2[0].x + aq2[0].y, aq2[1].x + aq2[1].y, aq2[2].x + aq2[2].y, aq2[3].x + aq2[3].y);
                }
                float4 *red4 = reinterpret_cast<float4 *>(sl + oRED);
                if (kDelta) red4[(rl * 2 + 0) * C4 + c4] = ak;
                red4[(rl * 2 + 1) * C4 + c4] = aq;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(stream_done + 8u * (it & (NS - 1)));
        }
    } else {
        // ================= scalar groups ==========================================================
        // Two groups of four warps split the non-streaming work of every unit by function, so that
        // the preparation of unit i+1 runs beside the epilogue of unit i:
        //   prep group      cumulative decay, decayed multipliers (-> stream group), key-side replay
        //                   coefficients and q.k (-> epilogue group);
        //   epilogue group  cross-warp reduction, value-side replay, b, output, append.
        constexpr int kHalf = kGroupWarps / 2;
        const bool is_prep = warp < kGroupWarps + kHalf;
        const int gtid = tid - kPipeConsumers - (is_prep ? 0 : 32 * kHalf), gwarp = gtid >> 5;
        bool alive = true;
        if (is_prep) {
            for (int j = 0; j < n_items; ++j) {
                const int stg = j % NA;
                bool got = bounded_wait(full_aux + 8u * stg, (uint32_t)(j / NA) & 1u, abort_flag);
                got = got && bounded_wait(slot_free + 8u * (j & (NS - 1)), ((uint32_t)(j >> SH) & 1u) ^ 1u, abort_flag);
                if (group_any(!got, 1)) {
                    alive = false;
                    break;
                }
                const unsigned char *stage = aux_ring + (size_t)stg * lay.bytes;
                float *sl = slot_ptr(j);
                const int4 meta = *reinterpret_cast<const int4 *>(stage + lay.meta);
                const int len = meta.x, flags = meta.y;
                if (flags == 0) {
                    const IO *q_a = reinterpret_cast<const IO *>(stage + lay.q);
                    const IO *k_a = reinterpret_cast<const IO *>(stage + lay.k);
                    const IO *K_a = reinterpret_cast<const IO *>(stage + lay.K);
                    const float *L_a = reinterpret_cast<const float *>(stage + lay.L);
                    const float *g_a = reinterpret_cast<const float *>(stage + lay.g);
                    const float *bonus_a = reinterpret_cast<const float *>(stage + lay.bonus);
                    float *q_s = sl + oQ, *k_s = sl + oK, *lbar_s = sl + oLB;
                    if (gtid < D) {
                        const float qv = to_f32(q_a[gtid]);
                        const float kv = to_f32(k_a[gtid]);
                        const float lold = (len > 0) ? L_a[(len - 1) * DL + (kVecDecay ? gtid : 0)] : 0.f;
                        const float lnew = lold + (kVecDecay ? g_a[gtid] : __int_as_float(meta.z));
                        q_s[gtid] = qv;
                        k_s[gtid] = kv;
                        lbar_s[gtid] = kPost ? lnew : lold;  // the decay level the readouts refer to
                        sl[oLN + gtid] = lnew;                // the level stored with the appended entry
                        const float e = expf(kPost ? lnew : lold);
                        sl[oMK + gtid] = e * kv;
                        sl[oMQ + gtid] = e * qv;
                    }
                    if (gtid == 0) sl[oSC + 1] = __int_as_float(0);
                    group_sync(1);
                    if (gtid == 0) mbar_arrive(prep_done + 8u * (j & (NS - 1)));  // the stream group may start on this unit

                    // Key-side replay coefficients, sixteen entries per round of the group: eight lanes share an
                    // entry (a lane takes 2 x 8 key channels with 16-byte loads), a warp pass covers four entries
                    // and the sums are combined in three shuffle rounds.  (With a whole warp per entry -- eight
                    // entries per round, five shuffle rounds -- the launch time climbed in steps at 9, 17, 25 live
                    // entries: from the second round on this group was the slowest stage.)
                    {
                        const int s8 = lane & 7, e4 = lane >> 3;
                        for (int i0 = 4 * gwarp; i0 < len; i0 += 4 * kHalf) {
                            const int i = i0 + e4;
                            float dq = 0.f, dk = 0.f;
                            if (i < len) {
#pragma unroll
                                for (int hh = 0; hh < D / 64; ++hh) {
                                    const int ch = 8 * s8 + 64 * hh;
                                    float q8[8], k8[8], ke[8];
                                    load8(q_s + ch, q8);
                                    if (kDelta) load8(k_s + ch, k8);
                                    load8(K_a + i * D + ch, ke);
                                    if (kVecDecay) {
                                        float lb8[8], le[8];
                                        load8(lbar_s + ch, lb8);
                                        load8(L_a + i * D + ch, le);
#pragma unroll
                                        for (int e = 0; e < 8; ++e) ke[e] *= expf(lb8[e] - le[e]);
                                    }
#pragma unroll
                                    for (int e = 0; e < 8; ++e) {
                                        dq = fmaf(q8[e], ke[e], dq);
                                        if (kDelta) dk = fmaf(k8[e], ke[e], dk);
                                    }
                                }
                            }
#pragma unroll
                            for (int o = 1; o < 8; o <<= 1) {
                                dq += __shfl_xor_sync(0xffffffffu, dq, o);
                                if (kDelta) dk += __shfl_xor_sync(0xffffffffu, dk, o);
                            }
                            if (s8 == 0 && i < len) {
                                const float w = kVecDecay ? 1.f : expf(lbar_s[0] - L_a[i]);
                                sl[oCQ + i] = w * dq;
                                if (kDelta) sl[oCK + i] = w * dk;
                            }
                        }
                    }
                    float qv[EPL], kv[EPL];
                    load_vec<float, EPL>(q_s + lane * EPL, qv);
                    load_vec<float, EPL>(k_s + lane * EPL, kv);
                    if (gwarp == kHalf - 1) {  // q.k for the delta rule, r.(bonus.k) for RWKV6
                        float d = 0.f;
                        float bw[EPL];
                        if (!kPost) load_vec<float, EPL>(bonus_a + lane * EPL, bw);
#pragma unroll
                        for (int e = 0; e < EPL; ++e) d = fmaf(kPost ? qv[e] : qv[e] * bw[e], kv[e], d);
                        d = warp_sum(d);
                        if (lane == 0) sl[oSC] = d;
                    }
                } else if (gtid == 0) {
                    sl[oSC + 1] = __int_as_float(flags);
                    mbar_arrive(prep_done + 8u * (j & (NS - 1)));
                }
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(coef_done + 8u * (j & (NS - 1)));  // this warp's coefficients are in the slot
                    mbar_arrive(empty_aux + 8u * stg);      // ... and it is done with the unit's aux stage
                }
            }
        } else {
            for (int it = 0; it < n_items; ++it) {
                const int stg = it % NA;
                const uint32_t par = (uint32_t)(it >> SH) & 1u;
                bool got = bounded_wait(stream_done + 8u * (it & (NS - 1)), par, abort_flag);
                got = got && bounded_wait(coef_done + 8u * (it & (NS - 1)), par, abort_flag);
                got = got && bounded_wait(full_aux + 8u * stg, (uint32_t)(it / NA) & 1u, abort_flag);
                if (group_any(!got, 2)) {
                    alive = false;
                    break;
                }
                const unsigned char *stage = aux_ring + (size_t)stg * lay.bytes;
                const int4 meta = *reinterpret_cast<const int4 *>(stage + lay.meta);
                const int len = meta.x, flags = meta.y;
                if (flags == 0 && gtid < D) {  // this thread owns output column c: both readouts, b, the output
                    const int slot = *reinterpret_cast<const int *>(stage + lay.meta + 16);
                    const int item = first + it * stride;
                    const size_t unit = (size_t)slot * H + item % H;
                    const IO *k_a = reinterpret_cast<const IO *>(stage + lay.k);
                    const IO *v_a = reinterpret_cast<const IO *>(stage + lay.v);
                    const UL *U_a = reinterpret_cast<const UL *>(stage + lay.U);
                    const float *sl = slot_ptr(it);
                    const float *red_s = sl + oRED;
                    const int c = gtid;
                    float yk = 0.f, yq = 0.f;
#pragma unroll
                    for (int r = 0; r < RL; ++r) {
                        if (kDelta) yk += red_s[(r * 2 + 0) * D + c];
                        yq += red_s[(r * 2 + 1) * D + c];
                    }
#pragma unroll 4
                    for (int i = 0; i < len; ++i) {
                        const float u = to_f32(U_a[i * D + c]);
                        if (kDelta) yk = fmaf(sl[oCK + i], u, yk);
                        yq = fmaf(sl[oCQ + i], u, yq);
                    }
                    const IO v_raw = v_a[c];
                    UL *Uout = static_cast<UL *>(st.U_log) + (unit * cap + len) * D;
                    IO *og = static_cast<IO *>(tk.out) + (size_t)item * D;
                    // the new entry is read again by the following steps: same L2 policy as the log's reads
                    const uint64_t keep = l2_policy_keep(st.keep_fraction(len + 1, total, kEntryBytes));
                    if (kDelta) {
                        const float bval = __int_as_float(meta.w) * (to_f32(v_raw) - yk);
                        st_hint(Uout + c, from_f32<UL>(bval), keep);
                        og[c] = from_f32<IO>(st.scale * fmaf(sl[oSC], bval, yq));
                    } else {
                        st_hint(Uout + c, from_f32<UL>(to_f32(v_raw)), keep);  // lossless: U log dtype equals the I/O dtype
                        og[c] = from_f32<IO>((kPost ? st.scale : 1.f) * fmaf(sl[oSC], to_f32(v_raw), yq));
                    }
                    st_hint(static_cast<IO *>(st.K_log) + (unit * cap + len) * D + c, k_a[c], keep);
                    if (kVecDecay) st_hint(st.decay_log + (unit * cap + len) * DL + c, sl[oLN + c], keep);
                    if (c == 0) {
                        if (!kVecDecay) st_hint(st.decay_log + unit * cap + len, sl[oLN], keep);
                        st.log_len[unit] = len + 1;
                    }
                }
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(slot_free + 8u * (it & (NS - 1)));  // the prep group may reuse the hand-over slot
                    mbar_arrive(empty_aux + 8u * stg);       // this warp is done with the unit's aux stage
                }
            }
        }
        if (!alive && gtid == 0 && st.status) atomicOr(st.status, DELTALOG_STATUS_TIMEOUT);
    }
}

}  // namespace deltalog
