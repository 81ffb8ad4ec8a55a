// The fused merge step (Algorithm 1, else-branch; Eq. 5 with the current-token term a_t b_t^T) as a
// resident CTA that walks over its share of the (batch row, head) units with the next unit's operands
// in flight.
//
// The arithmetic, the thread mapping (a thread owns NP consecutive rows x 4 columns of the tile in
// registers) and the order of operations are those of decode_merge_step_kernel.  What differs is
// where a unit's operands come from.  With one unit per CTA, a CTA's life is one chain -- request the
// tile, wait, weights, rank update, readouts, reduction, b, store, exit -- and while it computes and
// stores, nothing of it is in flight; two such CTAs fit an SM (the tile takes 64 registers of each
// thread).  Here the tile of unit n+1 is requested with one bulk copy into a shared-memory buffer as
// soon as unit n's tile has been moved from that buffer into registers, and the log and the token
// vectors of unit n+1 as soon as unit n has consumed its own (raw key-side rows and token after the
// weights are formed, value-side rows after the rank update), so every operand of a unit has a
// unit's compute and store time to arrive and the only wait left is a short one for the tile.
// Measured per launch against one unit per CTA at capacity 16: configuration 1's shape 114 -> 110-113 us
// (capacity 8: 101 -> 88 us), configuration 2's 266 -> 222 us, configuration 3's 144 -> 125 us; the launcher
// uses it up to capacity 16.  (The plain merge, whose CTAs have no readout /
// reduction chain to hide, does not gain: one unit per CTA already runs at 0.96 of the copy peak
// there and this scheme was 5-10 % behind it, so the merge keeps merge_kernel.)
//
// The rank update uses scalar FMAs: two CTAs that stay on an SM for the whole launch share the
// packed-FMA pipe badly (the older CTA's warps are served first; the younger CTA's rank update took
// 13 us instead of 4 until the older one had finished), while scalar FMAs are shared evenly.
//
// Shared memory per CTA: one tile buffer, one raw copy of a log (K, Lambda, U as stored), one raw
// token, the weights A, the partial readouts and the small vectors -- about 100 KB at head size 128
// and capacity 16, two CTAs per SM.  The wait for the tile's mbarrier is bounded in time like every
// wait of the library (DELTALOG_STATUS_TIMEOUT).
#pragma once

#include "common.cuh"
#include "decode_pipelined.cuh"  // mbarrier / bulk-copy primitives and the bounded wait

namespace deltalog {

template <int OP, int DK, int DV, typename IO, typename UL, typename BT>
struct FusedResidentLayout {
    static constexpr bool kVec = OpTraits<OP>::kVecDecay;
    static constexpr int DL = kVec ? DK : 1;
    static constexpr int NT = mat_threads<DK, DV>();
    static constexpr int RL = NT / (DV / 4);
    static constexpr int kTileBytes = DK * DV * (int)sizeof(BT);
    int tile, A, U, K, L, q, k, v, g, vec, red, bytes;  // byte offsets
    __host__ __device__ explicit FusedResidentLayout(int cap) {
        int o = 128;  // the mbarrier and the abort flags
        tile = o, o += kTileBytes;
        A = o, o += cap * DK * 4;                              // e^{lref_j - Lambda_ij} K_ij, fp32
        U = o, o += align_up(cap * DV * (int)sizeof(UL), 16);  // as stored
        K = o, o += align_up(cap * DK * (int)sizeof(IO), 16);  // as stored
        L = o, o += align_up(cap * DL * 4, 16);                // as stored
        q = o, o += DK * (int)sizeof(IO);
        k = o, o += DK * (int)sizeof(IO);
        v = o, o += DV * (int)sizeof(IO);
        g = o, o += kVec ? DK * 4 : 0;
        vec = o, o += (4 * DK + 2 * DV + 4) * 4;               // e, q, k, w [DK]; b, v [DV]; scalars
        red = o, o += 2 * DV * RL * 4;                         // partial readouts [RL][2][DV]
        bytes = align_up(o, 128);
    }
};

template <int OP, int DK, int DV, typename IO, typename UL, typename BT = float>
__global__ void __launch_bounds__(mat_threads<DK, DV>(), mat_threads<DK, DV>() <= 128 ? 4 : 2)
fused_step_resident_kernel(StateArgs st, TokenArgs tk, int32_t n_pairs, int32_t test_drop_pair) {
    using Lay = FusedResidentLayout<OP, DK, DV, IO, UL, BT>;
    constexpr bool kDelta = OpTraits<OP>::kDeltaRule;
    constexpr bool kPost = OpTraits<OP>::kPostReadout;
    constexpr bool kVecDecay = OpTraits<OP>::kVecDecay;
    constexpr int DL = Lay::DL, NT = Lay::NT, RL = Lay::RL;
    constexpr int C4 = DV / 4, NP = DK / RL, EPL = DK / 32;
    constexpr int kTileBytes = Lay::kTileBytes;
    constexpr int kPiece = kTileBytes < kChunkBytes ? kTileBytes : kChunkBytes, kPieces = kTileBytes / kPiece;
    static_assert(NT >= DK && NT >= (kDelta ? 2 : 1) * DV, "one thread per key channel and per output column");
    static_assert(kPieces <= 32 && kPieces * kPiece == kTileBytes, "a tile is a whole number of pieces");

    extern __shared__ __align__(128) unsigned char smem[];
    const Lay lay(st.cap);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cap = st.cap, H = st.H;
    const uint32_t bar = smem_addr(smem);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + 16);
    const BT *T = reinterpret_cast<const BT *>(smem + lay.tile);
    float *A_s = reinterpret_cast<float *>(smem + lay.A);
    UL *U_raw = reinterpret_cast<UL *>(smem + lay.U);
    IO *K_raw = reinterpret_cast<IO *>(smem + lay.K);
    float *L_raw = reinterpret_cast<float *>(smem + lay.L);
    IO *q_raw = reinterpret_cast<IO *>(smem + lay.q), *k_raw = reinterpret_cast<IO *>(smem + lay.k);
    IO *v_raw = reinterpret_cast<IO *>(smem + lay.v);
    float *g_raw = reinterpret_cast<float *>(smem + lay.g);
    float *e_s = reinterpret_cast<float *>(smem + lay.vec);   // [DK] e^{lref}
    float *q_s = e_s + DK, *k_s = q_s + DK, *w_s = k_s + DK;  // w: RWKV6's e^{lambda_t}
    float *b_s = w_s + DK, *v_s = b_s + DV, *scal_s = v_s + DV;  // scal[0] = q.k  (or r.(bonus.k))
    float *red_s = reinterpret_cast<float *>(smem + lay.red);

    if (tid == 0) {
        mbar_init(bar, 1);
        abort_flag[0] = 0;
        abort_flag[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
    }
    __syncthreads();

    // pair (batch row * H + head) -> unit (slot * H + head), or -1 for a padding row and a slot outside the pool
    auto unit_of = [&](int pair) -> int {
        if (pair < 0) return -1;
        int slot;
        if (!resolve_slot(tk.slot_idx, pair / H, st.num_slots, st.status, tid, slot)) return -1;
        return slot * H + pair % H;
    };
    // (Test builds only, DELTALOG_TEST_HOOKS: the tile of pair test_drop_pair is never requested, so that the wait
    // for it runs out -- the way to see the give-up path without hanging or faulting anything.)
    auto request_tile = [&](int unit, int pair) {
#if DELTALOG_TEST_HOOKS
        if (pair == test_drop_pair) return;
#endif
        if (warp == 0) {
            if (lane == 0) mbar_arrive_expect_tx(bar, kTileBytes);
            __syncwarp();
            if (lane < kPieces)
                bulk_copy_g2s(smem_addr(T) + lane * kPiece,
                              static_cast<const char *>(st.S_base) + (size_t)unit * kTileBytes + lane * kPiece, kPiece, bar);
        }
    };
    auto request_key_side = [&](int unit, int pair) {  // raw key rows, snapshots, and the token's vectors
        cta_cp_async(K_raw, static_cast<const IO *>(st.K_log) + (size_t)unit * cap * DK, cap * DK * (int)sizeof(IO), tid, NT);
        cta_cp_async(L_raw, st.decay_log + (size_t)unit * cap * DL, cap * DL * 4, tid, NT);
        const size_t qk = tk.qk_row(pair / H, pair % H);
        cta_cp_async(q_raw, static_cast<const IO *>(tk.q) + qk * DK, DK * (int)sizeof(IO), tid, NT);
        cta_cp_async(k_raw, static_cast<const IO *>(tk.k) + qk * DK, DK * (int)sizeof(IO), tid, NT);
        cta_cp_async(v_raw, static_cast<const IO *>(tk.v) + (size_t)pair * DV, DV * (int)sizeof(IO), tid, NT);
        if (kVecDecay && tk.g) cta_cp_async(g_raw, tk.g + (size_t)pair * DK, DK * 4, tid, NT);
    };
    auto request_value_side = [&](int unit) {
        cta_cp_async(U_raw, static_cast<const UL *>(st.U_log) + (size_t)unit * cap * DV, cap * DV * (int)sizeof(UL), tid, NT);
    };
    // per-unit scalars: every thread reads the same words
    auto scalars_of = [&](int unit, int pair, int &len, float &beta, float &gsc) {
        len = st.log_len[unit];
        beta = kDelta ? tk.beta[pair] : 0.f;
        gsc = (!kVecDecay && tk.g) ? tk.g[pair] : 0.f;  // no gate: plain linear attention
    };

    // Pairs are taken from the last to the first: the tiles written last (still in L2 when the kernel ends) are
    // then the ones the next decode step, which walks upwards from pair 0, reads first.
    int pair = n_pairs - 1 - (int)blockIdx.x;
    int unit = unit_of(pair);
    int len = 0;
    float beta = 0.f, gsc = 0.f;
    if (unit >= 0) {
        request_tile(unit, pair);
        request_key_side(unit, pair);
        request_value_side(unit);
        scalars_of(unit, pair, len, beta, gsc);
    }
    cp_async_commit();

    const int c4 = tid % C4, rl = tid / C4;
    uint32_t phase = 0;
    bool timed_out = false;
    for (; pair >= 0; pair -= gridDim.x) {
        const int npair = pair - (int)gridDim.x;
        const int nunit = unit_of(npair);
        float bonus_r[EPL];
#pragma unroll
        for (int e = 0; e < EPL; ++e)
            bonus_r[e] = (!kPost && warp == 0) ? tk.u_bonus[(size_t)(pair % H) * DK + lane + 32 * e] : 1.f;

        // ---- the tile: shared memory -> registers --------------------------------------------------
        float4 s[NP];
        if (unit >= 0) {
            if (!bounded_wait(bar, phase, abort_flag)) timed_out = true;
            phase ^= 1u;
#pragma unroll
            for (int p = 0; p < NP; ++p) s[p] = base_load4<BT>(T + ((size_t)(rl * NP + p) * C4 + c4) * 4);
        }
        cp_async_wait_all();
        __syncthreads();  // (A) the tile buffer is free; this unit's raw log and token are visible to all
        if (abort_flag[0]) break;
        int nlen = 0;
        float nbeta = 0.f, ngsc = 0.f;
        if (nunit >= 0) {
            request_tile(nunit, npair);
            scalars_of(nunit, npair, nlen, nbeta, ngsc);
        }
        if (unit < 0) {  // padding row: nothing to do but to pass the requests on
            if (nunit >= 0) {
                request_key_side(nunit, npair);
                request_value_side(nunit);
            }
            cp_async_commit();
            unit = nunit, len = nlen, beta = nbeta, gsc = ngsc;
            continue;
        }
        len = len < 0 ? 0 : (len > cap ? cap : len);

        // ---- key-side weights A_ij = e^{lref_j - Lambda_ij} K_ij ------------------------------------
        // lref: the decay level the state is materialised at -- lbar' = lbar + lambda_t for the delta rule and the
        // additive operators (both readouts are taken on the decayed state), lbar for RWKV6 (readout on the
        // pre-update state).
        const float *lold = L_raw + (size_t)(len > 0 ? len - 1 : 0) * DL;
        for (int x = tid * 4; x < len * DK; x += NT * 4) {
            const int i = x / DK, j = x % DK;
            float kv[4], w[4];
            load_vec<IO, 4>(K_raw + x, kv);
            if (kVecDecay) {
                const float4 lo = *reinterpret_cast<const float4 *>(lold + j);
                const float4 li = *reinterpret_cast<const float4 *>(L_raw + (size_t)i * DK + j);
                float4 gl = make_float4(0.f, 0.f, 0.f, 0.f);
                if (kPost && tk.g) gl = *reinterpret_cast<const float4 *>(g_raw + j);
                w[0] = expf(lo.x + gl.x - li.x), w[1] = expf(lo.y + gl.y - li.y);
                w[2] = expf(lo.z + gl.z - li.z), w[3] = expf(lo.w + gl.w - li.w);
            } else {
                w[0] = w[1] = w[2] = w[3] = expf(lold[0] + gsc - L_raw[i]);  // (len > 0 here)
            }
            *reinterpret_cast<float4 *>(A_s + x) = make_float4(w[0] * kv[0], w[1] * kv[1], w[2] * kv[2], w[3] * kv[3]);
        }
        if (tid < DK) {
            const float lo = len > 0 ? lold[kVecDecay ? tid : 0] : 0.f;
            const float lam = kVecDecay ? (tk.g ? g_raw[tid] : 0.f) : gsc;
            q_s[tid] = to_f32(q_raw[tid]);
            k_s[tid] = to_f32(k_raw[tid]);
            e_s[tid] = expf(kPost ? lo + lam : lo);
            w_s[tid] = expf(lam);
        }
        if (tid < DV) v_s[tid] = to_f32(v_raw[tid]);
        __syncthreads();  // (B) the raw key-side rows and the raw token have been consumed
        if (nunit >= 0) request_key_side(nunit, npair);
        cp_async_commit();

        if (warp == 0) {  // q.k for the delta rule, r.(bonus.k) for RWKV6
            float d = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) {
                const int j = lane + 32 * e;
                d = fmaf(q_s[j] * bonus_r[e], k_s[j], d);
            }
            d = warp_sum(d);
            if (lane == 0) scal_s[0] = d;
        }

        // ---- materialise at lref (Eq. 6) in registers ----------------------------------------------
#pragma unroll
        for (int p = 0; p < NP; ++p) {
            const float e = e_s[rl * NP + p];
            s[p] = make_float4(e * s[p].x, e * s[p].y, e * s[p].z, e * s[p].w);
        }
        rank_update_scalar<NP>(
            s, len,
            [&](int i, int p4) { return reinterpret_cast<const float4 *>(A_s + (size_t)i * DK + rl * NP)[p4]; },
            [&](int i) {
                float uv[4];
                load_vec<UL, 4>(U_raw + (size_t)i * DV + 4 * c4, uv);
                return make_float4(uv[0], uv[1], uv[2], uv[3]);
            });

        // ---- the two readouts from the materialised tile --------------------------------------------
        float4 ak = make_float4(0.f, 0.f, 0.f, 0.f), aq = ak;
#pragma unroll
        for (int p = 0; p < NP; ++p) {
            const int r = rl * NP + p;
            if (kDelta) ak = fma4(k_s[r], s[p], ak);
            aq = fma4(q_s[r], s[p], aq);
        }
        float4 *red4 = reinterpret_cast<float4 *>(red_s);
        if (kDelta) red4[(rl * 2 + 0) * C4 + c4] = ak;
        red4[(rl * 2 + 1) * C4 + c4] = aq;
        __syncthreads();  // (C) the weights and the raw value-side rows have been consumed
        if (nunit >= 0) request_value_side(nunit);
        cp_async_commit();

        const int which = tid / DV, c = tid % DV;  // which: 0 -> S'^T k half, 1 -> S'^T q half
        const bool active = kDelta ? (tid < 2 * DV) : (tid < DV);
        const int sel = kDelta ? which : 1;
        float y = 0.f;
        if (active) {
#pragma unroll
            for (int r = 0; r < RL; ++r) y += red_s[(r * 2 + sel) * DV + c];
        }
        IO *og = static_cast<IO *>(tk.out) + (size_t)pair * DV;
        if (kDelta) {
            if (tid < DV) b_s[c] = beta * (v_s[c] - y);
            __syncthreads();
            if (active && which == 1) og[c] = from_f32<IO>(st.scale * fmaf(scal_s[0], b_s[c], y));
        } else {
            if (active) {
                const float vv = v_s[c];  // (active threads are the first DV: c == tid)
                b_s[c] = vv;
                og[c] = from_f32<IO>((kPost ? st.scale : 1.f) * fmaf(scal_s[0], vv, y));
            }
            __syncthreads();
        }

        // ---- Eq. 5: the represented state plus the current update, written once; the log is cleared ----
        BT *Sg = static_cast<BT *>(st.S_base) + (size_t)unit * DK * DV;
        const float4 b4 = reinterpret_cast<const float4 *>(b_s)[c4];
#pragma unroll
        for (int p = 0; p < NP; ++p) {
            const int r = rl * NP + p;
            float4 x = s[p];
            if (!kPost) {
                const float a = w_s[r];
                x = make_float4(a * x.x, a * x.y, a * x.z, a * x.w);
            }
            base_store4<BT>(Sg + ((size_t)r * C4 + c4) * 4, fma4(k_s[r], b4, x));
        }
        if (tid == 0) st.log_len[unit] = 0;
        unit = nunit, len = nlen, beta = nbeta, gsc = ngsc;
    }
    cp_async_wait_all();
    if (abort_flag[0] && tid == 0) {
        // A wait ran out: report it, and give a tile copy that may still be in flight a (bounded) chance to land
        // before the CTA's shared memory is released.
        if (st.status) atomicOr(st.status, DELTALOG_STATUS_TIMEOUT);
        if (!timed_out) bounded_wait(bar, phase, abort_flag + 1);
    }
}

}  // namespace deltalog
