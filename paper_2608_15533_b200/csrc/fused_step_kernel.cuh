// Fused merge step: one CTA per (batch row, head) consumes a token AND materialises the state
// (Algorithm 1, else-branch; Eq. 5 with the current-token term a_t b_t^T), whatever the live length:
//
//   lbar  = Lambda[len-1] (0 if the log is empty),  lbar' = lbar + lambda_t
//   delta ops:  S'  = D(lbar') S_base + sum_i D(lbar' - Lambda[i]) K[i] U[i]^T      (decayed state)
//               b   = beta (v - S'^T k);  out = scale (S'^T q + (q.k) b);  S_base <- S' + k b^T
//   RWKV6:      S-  = D(lbar) S_base + sum_i D(lbar - Lambda[i]) K[i] U[i]^T        (pre-update state)
//               out = S-^T r + (r.(bonus.k)) v;                 S_base <- D(lambda_t) S- + k v^T
//   len <- 0   (lbar is Lambda[len-1], so clearing the length clears it too)
//
// One read and one write of the tile, like the eager step, plus one read of the live log.  The tile
// is requested first and held in registers: every thread owns NP consecutive rows x 4 columns.
#pragma once

#include "common.cuh"

namespace deltalog {

template <int DK, int DV, typename IO, typename UL>
__host__ __device__ constexpr size_t fused_step_smem_bytes(int cap, bool vec_decay) {
    constexpr int RL = mat_threads<DK, DV>() / (DV / 4);
    // A [cap][DK], U [cap][DV], e, q, k, w, lambda [DK] each, b [DV], partial sums [RL][2][DV], scalars; then the log as
    // it is stored (requested ahead of the length word): K [cap][DK], Lambda [cap][d_lambda], U where not fp32
    return sizeof(float) * ((size_t)cap * (DK + DV) + 5 * DK + DV + 2 * DV * RL + 4) + sizeof(IO) * (size_t)cap * DK +
           sizeof(float) * (((size_t)cap * (vec_decay ? DK : 1) + 3) / 4 * 4) +
           (sizeof(UL) == 4 ? 0 : sizeof(UL) * (size_t)cap * DV);
}

template <int OP, int DK, int DV, typename IO, typename UL, typename BT = float>
__global__ void __launch_bounds__(mat_threads<DK, DV>(), mat_threads<DK, DV>() <= 128 ? 4 : 2) decode_merge_step_kernel(StateArgs st, TokenArgs tk) {
    constexpr bool kDelta = OpTraits<OP>::kDeltaRule;
    constexpr bool kPost = OpTraits<OP>::kPostReadout;
    constexpr bool kVecDecay = OpTraits<OP>::kVecDecay;
    constexpr int DL = kVecDecay ? DK : 1;
    constexpr int NT = mat_threads<DK, DV>();
    constexpr int C4 = DV / 4, RL = NT / C4, NP = DK / RL, EPL = DK / 32;
    static_assert(NT >= DK && NT >= (kDelta ? 2 : 1) * DV, "one thread per key channel and per output column");

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // (pairs from the last to the first, see merge_kernel: what is written last is what the next decode step reads first)
    const int pair = gridDim.x - 1 - blockIdx.x;
    const int b = pair / st.H, h = pair % st.H;
    int slot;
    if (!resolve_slot(tk.slot_idx, b, st.num_slots, st.status, tid, slot)) return;
    const size_t unit = (size_t)slot * st.H + h, row = (size_t)b * st.H + h;
    const int cap = st.cap;

    BT *Sg = static_cast<BT *>(st.S_base) + unit * DK * DV;
    const int c4 = tid % C4, rl = tid / C4;
    float4 s[NP];
#pragma unroll
    for (int p = 0; p < NP; ++p) s[p] = base_load4<BT>(Sg + ((size_t)(rl * NP + p) * C4 + c4) * 4);
    // The token's vectors are requested here as well, into registers: nothing below waits for global memory
    // a second time (a CTA's run time is one chain of dependent round trips).
    const float *gg = tk.g + row * (kVecDecay ? DK : 1);
    const IO *vg = static_cast<const IO *>(tk.v) + row * DV;
    // (Measured on the same box: GDN shape 123 -> 113 us, RWKV6 shape unchanged, KDA shape 252 -> 262 us.)
    float q_r = 0.f, k_r = 0.f, lam_r = 0.f, v_r = 0.f, beta_r = 0.f, bonus_r[EPL];
    if (tid < DK) {
        q_r = to_f32(static_cast<const IO *>(tk.q)[tk.qk_row(b, h) * DK + tid]);
        k_r = to_f32(static_cast<const IO *>(tk.k)[tk.qk_row(b, h) * DK + tid]);
    }
    if (tid < DK || !kVecDecay) lam_r = tk.g ? gg[kVecDecay ? tid : 0] : 0.f;  // no gate: plain linear attention
    if (tid < DV) v_r = to_f32(vg[tid]);
    if (kDelta) beta_r = tk.beta[row];
#pragma unroll
    for (int e = 0; e < EPL; ++e) bonus_r[e] = (!kPost && warp == 0) ? tk.u_bonus[(size_t)h * DK + lane + 32 * e] : 1.f;

    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *A_s = reinterpret_cast<float *>(smem_raw);  // [len][DK]  e^{lref_j - Lambda_ij} K_ij
    float *U_s = A_s + (size_t)cap * DK;               // [len][DV]
    float *e_s = U_s + (size_t)cap * DV;               // [DK] e^{lref}
    float *q_s = e_s + DK;
    float *k_s = q_s + DK;
    float *w_s = k_s + DK;                             // RWKV6: e^{lambda_t}
    float *b_s = w_s + DK;                             // [DV]
    float *red_s = b_s + DV;                           // [RL][2][DV]
    float *scal_s = red_s + 2 * DV * RL;               // [0] = q.k  (or r.(bonus.k))
    float *lam_s = scal_s + 4;                         // [DK] the token's log-decay
    IO *K_raw = reinterpret_cast<IO *>(lam_s + DK);    // [cap][DK] as stored
    float *L_raw = reinterpret_cast<float *>(K_raw + (size_t)cap * DK);  // [cap][DL]
    UL *U_raw = sizeof(UL) == 4 ? reinterpret_cast<UL *>(U_s) : reinterpret_cast<UL *>(L_raw + ((size_t)cap * DL + 3) / 4 * 4);

    const IO *Kg = static_cast<const IO *>(st.K_log) + unit * cap * DK;
    const UL *Ug = static_cast<const UL *>(st.U_log) + unit * cap * DV;
    const float *Lg = st.decay_log + unit * cap * DL;
    // The whole log is requested (asynchronously, into shared memory) together with the tile, BEFORE the length
    // word is known: a CTA's run time is one chain of dependent memory round trips, and this takes one of them
    // out.  Entries beyond the live length are never used.  (Needs 16-byte aligned snapshot rows.)
    const bool ahead = kVecDecay || cap % 4 == 0;
    if (ahead) {
        cta_cp_async(K_raw, Kg, cap * DK * (int)sizeof(IO), tid, NT);
        cta_cp_async(U_raw, Ug, cap * DV * (int)sizeof(UL), tid, NT);
        cta_cp_async(L_raw, Lg, (cap * DL * 4 + 15) / 16 * 16, tid, NT);
        cp_async_commit();
    }
    int len = st.log_len[unit];
    len = len < 0 ? 0 : (len > cap ? cap : len);
    const float *lold = (ahead ? L_raw : Lg) + (size_t)(len > 0 ? len - 1 : 0) * DL;
    if (tid < DK) lam_s[tid] = lam_r;   // the token's log-decay per key channel, for the weights below
    if (ahead) {
        cp_async_wait_all();
        __syncthreads();
        for (int x = tid * 4; x < len * DK; x += NT * 4) {
            const int i = x / DK, j = x % DK;
            float kv[4], w[4];
            load_vec<IO, 4>(K_raw + x, kv);
            if (kVecDecay) {
                const float4 lo = *reinterpret_cast<const float4 *>(lold + j);
                const float4 li = *reinterpret_cast<const float4 *>(L_raw + (size_t)i * DK + j);
                float4 gl = make_float4(0.f, 0.f, 0.f, 0.f);
                if (kPost) gl = *reinterpret_cast<const float4 *>(lam_s + j);
                w[0] = expf(lo.x + gl.x - li.x), w[1] = expf(lo.y + gl.y - li.y);
                w[2] = expf(lo.z + gl.z - li.z), w[3] = expf(lo.w + gl.w - li.w);
            } else {
                const float lref = lold[0] + lam_s[0];  // (len > 0 here)
                w[0] = w[1] = w[2] = w[3] = expf(lref - L_raw[i]);
            }
            *reinterpret_cast<float4 *>(A_s + x) = make_float4(w[0] * kv[0], w[1] * kv[1], w[2] * kv[2], w[3] * kv[3]);
        }
        if (sizeof(UL) != 4) {
            for (int x = tid * 4; x < len * DV; x += NT * 4) {
                float uv[4];
                load_vec<UL, 4>(U_raw + x, uv);
                *reinterpret_cast<float4 *>(U_s + x) = make_float4(uv[0], uv[1], uv[2], uv[3]);
            }
        }
    } else
    // lref: the decay level the state is materialised at -- lbar' for the delta rule (both readouts
    // are taken on the decayed state), lbar for RWKV6 (readout on the pre-update state).
    if (!kVecDecay) {
        const float lref = (len > 0 ? lold[0] : 0.f) + lam_r;  // (scalar decay: every thread below DK holds it)
        for (int x = tid * 4; x < len * DK; x += NT * 4) {
            const float wi = expf(lref - Lg[x / DK]);
            float kv[4];
            load_vec<IO, 4>(Kg + x, kv);
            *reinterpret_cast<float4 *>(A_s + x) = make_float4(wi * kv[0], wi * kv[1], wi * kv[2], wi * kv[3]);
        }
        for (int x = tid * 4; x < len * DV; x += NT * 4) {
            float uv[4];
            load_vec<UL, 4>(Ug + x, uv);
            *reinterpret_cast<float4 *>(U_s + x) = make_float4(uv[0], uv[1], uv[2], uv[3]);
        }
    } else {
        for (int x = tid; x < len * DK; x += NT) {
            const int i = x / DK, j = x % DK;
            const float lref = lold[j] + (kPost ? gg[j] : 0.f);
            A_s[x] = expf(lref - Lg[(size_t)i * DK + j]) * to_f32(Kg[x]);
        }
        for (int x = tid; x < len * DV; x += NT) U_s[x] = to_f32(Ug[x]);
    }
    if (tid < DK) {
        const int jl = kVecDecay ? tid : 0;
        const float lo = len > 0 ? lold[jl] : 0.f;
        q_s[tid] = q_r;
        k_s[tid] = k_r;
        e_s[tid] = expf(kPost ? lo + lam_r : lo);
        w_s[tid] = expf(lam_r);
    }
    __syncthreads();

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

    // materialise at lref (Eq. 6) in registers
#pragma unroll
    for (int p = 0; p < NP; ++p) {
        const float e = e_s[rl * NP + p];
        s[p] = make_float4(e * s[p].x, e * s[p].y, e * s[p].z, e * s[p].w);
    }
    const float4 *U4 = reinterpret_cast<const float4 *>(U_s);
    rank_update<NP>(
        s, len,
        [&](int i, int p4) { return reinterpret_cast<const float4 *>(A_s + (size_t)i * DK + rl * NP)[p4]; },
        [&](int i) { return U4[i * C4 + c4]; });

    // the two readouts from the materialised tile
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
    __syncthreads();

    const int which = tid / DV, c = tid % DV;  // which: 0 -> S'^T k half, 1 -> S'^T q half
    const bool active = kDelta ? (tid < 2 * DV) : (tid < DV);
    const int sel = kDelta ? which : 1;
    float y = 0.f;
    if (active) {
#pragma unroll
        for (int r = 0; r < RL; ++r) y += red_s[(r * 2 + sel) * DV + c];
    }
    IO *og = static_cast<IO *>(tk.out) + row * DV;
    if (kDelta) {
        if (tid < DV) b_s[c] = beta_r * (v_r - y);
        __syncthreads();
        if (active && which == 1) og[c] = from_f32<IO>(st.scale * fmaf(scal_s[0], b_s[c], y));
    } else {
        if (active) {
            const float vv = v_r;   // (active threads are the first DV: c == tid)
            b_s[c] = vv;
            og[c] = from_f32<IO>((kPost ? st.scale : 1.f) * fmaf(scal_s[0], vv, y));
        }
        __syncthreads();
    }

    // Eq. 5: the represented state plus the current update, written once; the log is cleared
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
}

}  // namespace deltalog
