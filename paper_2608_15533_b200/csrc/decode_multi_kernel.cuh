// Multi-token decode + append: T consecutive tokens per row in one launch (the step a server takes
// when it verifies speculative tokens or feeds several tokens of one request at once).
//
// Exactly the arithmetic of T successive decode + append steps (Algorithm 1, append branch; Eq. 4 and
// Eq. 6) -- but the base tile is read from HBM ONCE for all T tokens and kept in registers, and the
// log grows in shared memory as the tokens are consumed.  One CTA per (batch row, head); token
// tensors are [B, T, H, d].  A row needs room for all T entries (len + T <= cap): otherwise nothing
// of it is processed and DELTALOG_STATUS_LOG_FULL is raised.
//
// Per token (lbar = Lambda[len-1] or 0, lbar' = lbar + lambda_t, len = entries so far):
//   delta rule:  y_k = S_base^T (e^{lbar'} . k) + sum_i ck_i U_i,  b = beta (v - y_k),
//                out = scale (S_base^T (e^{lbar'} . q) + sum_i cq_i U_i + (q.k) b)
//   b = v ops:   out = scale (y_q + (q.k) v)           RWKV6: readout at lbar, out = y_r + (r.(bonus.k)) v
//   append:      K[len] = k, U[len] = b, Lambda[len] = lbar'
#pragma once

#include "common.cuh"
#include "decode_kernel.cuh"

namespace deltalog {

template <int OP, int DK, int DV, typename IO, typename UL, typename BT = float>
__global__ void __launch_bounds__(decode_threads<DK, DV>(), decode_threads<DK, DV>() >= 256 ? 2 : 8)
decode_multi_kernel(StateArgs st, TokenArgs tk, int32_t T) {
    constexpr int NT = decode_threads<DK, DV>();
    constexpr int NW = NT / 32;
    constexpr bool kDelta = OpTraits<OP>::kDeltaRule;
    constexpr bool kPost = OpTraits<OP>::kPostReadout;
    constexpr bool kVecDecay = OpTraits<OP>::kVecDecay;
    constexpr int DL = kVecDecay ? DK : 1;
    constexpr int C4 = DV / 4, RL = NT / C4, NP = DK / RL, EPL = DK / 32;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.x / st.H, h = blockIdx.x % st.H;
    int slot;
    if (!resolve_slot(tk.slot_idx, b, st.num_slots, st.status, tid, slot)) return;
    const size_t unit = (size_t)slot * st.H + h;
    const int cap = st.cap;

    // ---- the base tile: one read for all T tokens ------------------------------------------------
    const BT *Sg = static_cast<const BT *>(st.S_base) + unit * DK * DV;
    const int c4 = tid % C4, rl = tid / C4;
    float4 s[NP];
#pragma unroll
    for (int p = 0; p < NP; ++p) s[p] = base_ldg4<BT>(Sg + ((size_t)(p * RL + rl) * C4 + c4) * 4);

    const int len0 = st.log_len[unit];
    if (len0 < 0 || len0 + T > cap) {  // no room for all T entries: the caller merges first
        if (tid == 0 && st.status) atomicOr(st.status, DELTALOG_STATUS_LOG_FULL);
        return;
    }

    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *q_s = reinterpret_cast<float *>(smem_raw);
    float *k_s = q_s + DK;
    float *mk_s = k_s + DK;     // e^{lbar'} . k
    float *mq_s = mk_s + DK;    // e^{lbar'} . q   (RWKV6: e^{lbar} . r)
    float *b_s = mq_s + DK;     // [DV]
    float *lold_s = b_s + DV;   // the decay level the readouts refer to
    float *ck_s = lold_s + DK;  // [kMaxCap]
    float *cq_s = ck_s + kMaxCap;
    float *red_s = cq_s + kMaxCap;           // [RL][2][DV]
    float *scal_s = red_s + 2 * DV * RL;     // [0] = q.k  (or r.(bonus.k))
    UL *U_s = reinterpret_cast<UL *>(scal_s + 4);
    IO *K_s = reinterpret_cast<IO *>(U_s + (size_t)cap * DV);
    float *Lam_s = reinterpret_cast<float *>(K_s + (size_t)cap * DK);

    // ---- the live log, staged once; it grows in shared memory below ------------------------------
    IO *Kg = static_cast<IO *>(st.K_log) + unit * cap * DK;
    UL *Ug = static_cast<UL *>(st.U_log) + unit * cap * DV;
    float *Lg = st.decay_log + unit * cap * DL;
    cta_cp_async(K_s, Kg, len0 * DK * (int)sizeof(IO), tid, NT);
    cta_cp_async(U_s, Ug, len0 * DV * (int)sizeof(UL), tid, NT);
    if (kVecDecay) cta_cp_async(Lam_s, Lg, len0 * DK * (int)sizeof(float), tid, NT);
    cp_async_commit();
    if (!kVecDecay && tid < len0) Lam_s[tid] = Lg[tid];
    cp_async_wait_all();
    __syncthreads();

    // The vectors of token t + 1 are requested while token t is being processed, so that their
    // latency hides behind its arithmetic (a thread holds the elements it will consume itself).
    struct Tok {
        IO q, k, v;
        float g, beta;
    };
    auto load_token = [&](int t) {
        Tok x;
        const size_t row = ((size_t)b * T + t) * st.H + h;                       // (batch row, token, head)
        const size_t row_qk = ((size_t)b * T + t) * tk.H_qk + h / tk.qk_group;
        const int c = tid % DV;
        x.q = x.k = from_f32<IO>(0.f);
        x.g = 0.f;
        x.beta = kDelta ? tk.beta[row] : 0.f;
        if (tid < DK) {
            x.q = static_cast<const IO *>(tk.q)[row_qk * DK + tid];
            x.k = static_cast<const IO *>(tk.k)[row_qk * DK + tid];
            x.g = tk.g ? tk.g[row * DL + (kVecDecay ? tid : 0)] : 0.f;
        }
        x.v = static_cast<const IO *>(tk.v)[row * DV + c];
        return x;
    };
    Tok nxt = load_token(0);
    for (int t = 0; t < T; ++t) {
        const int len = len0 + t;
        const size_t row = ((size_t)b * T + t) * st.H + h;
        const Tok cur = nxt;
        if (t + 1 < T) nxt = load_token(t + 1);
        IO k_raw = cur.k;
        float lnew = 0.f;
        if (tid < DK) {
            const float qv = to_f32(cur.q);
            const float kv = to_f32(k_raw);
            const float lold = (len > 0) ? Lam_s[(size_t)(len - 1) * DL + (kVecDecay ? tid : 0)] : 0.f;
            lnew = lold + cur.g;
            q_s[tid] = qv;
            k_s[tid] = kv;
            lold_s[tid] = kPost ? lnew : lold;
            const float e = expf(kPost ? lnew : lold);
            mk_s[tid] = e * kv;
            mq_s[tid] = e * qv;
        }
        __syncthreads();

        // key-side replay coefficients: one warp per live entry
        for (int i = warp; i < len; i += NW) {
            float dq = 0.f, dk = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) {
                const int j = lane + 32 * e;
                float kij = to_f32(K_s[i * DK + j]);
                if (kVecDecay) kij *= expf(lold_s[j] - Lam_s[i * DK + j]);
                dq = fmaf(q_s[j], kij, dq);
                if (kDelta) dk = fmaf(k_s[j], kij, dk);
            }
            dq = warp_sum(dq);
            if (kDelta) dk = warp_sum(dk);
            if (lane == 0) {
                const float w = kVecDecay ? 1.f : expf(lold_s[0] - Lam_s[i]);
                cq_s[i] = w * dq;
                if (kDelta) ck_s[i] = w * dk;
            }
        }
        if (warp == NW - 1) {  // q.k, or r.(bonus.k) for RWKV6
            float d = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) {
                const int j = lane + 32 * e;
                const float w = kPost ? 1.f : tk.u_bonus[(size_t)h * DK + j];
                d = fmaf(q_s[j] * w, k_s[j], d);
            }
            d = warp_sum(d);
            if (lane == 0) scal_s[0] = d;
        }

        // base pass from the registers
        float4 ak = make_float4(0.f, 0.f, 0.f, 0.f), aq = ak;
#pragma unroll
        for (int p = 0; p < NP; ++p) {
            const int r = p * RL + rl;
            if (kDelta) ak = fma4(mk_s[r], s[p], ak);
            aq = fma4(mq_s[r], s[p], aq);
        }
        float4 *red4 = reinterpret_cast<float4 *>(red_s);
        if (kDelta) red4[(rl * 2 + 0) * C4 + c4] = ak;
        red4[(rl * 2 + 1) * C4 + c4] = aq;
        __syncthreads();

        // reduce, value-side replay, b, output, append (shared memory and global)
        const int which = tid / DV, c = tid % DV;
        const bool active = kDelta ? (tid < 2 * DV) : (tid < DV);
        const int sel = kDelta ? which : 1;
        float y = 0.f;
        if (active) {
#pragma unroll
            for (int r = 0; r < RL; ++r) y += red_s[(r * 2 + sel) * DV + c];
            const float *coef = sel ? cq_s : ck_s;
            for (int i = 0; i < len; ++i) y = fmaf(coef[i], to_f32(U_s[i * DV + c]), y);
        }
        IO *og = static_cast<IO *>(tk.out) + row * DV;
        if (kDelta) {
            if (tid < DV) {
                const float bval = cur.beta * (to_f32(cur.v) - y);
                b_s[c] = bval;
                const UL bu = from_f32<UL>(bval);
                U_s[(size_t)len * DV + c] = bu;
                Ug[(size_t)len * DV + c] = bu;
            }
            __syncthreads();
            if (active && which == 1) og[c] = from_f32<IO>(st.scale * fmaf(scal_s[0], b_s[c], y));
        } else if (active) {
            const IO v_raw = cur.v;
            og[c] = from_f32<IO>((kPost ? st.scale : 1.f) * fmaf(scal_s[0], to_f32(v_raw), y));
            const UL bu = from_f32<UL>(to_f32(v_raw));
            U_s[(size_t)len * DV + c] = bu;
            Ug[(size_t)len * DV + c] = bu;
        }
        if (tid < DK) {
            K_s[(size_t)len * DK + tid] = k_raw;
            Kg[(size_t)len * DK + tid] = k_raw;
            if (kVecDecay) {
                Lam_s[(size_t)len * DK + tid] = lnew;
                Lg[(size_t)len * DK + tid] = lnew;
            }
        }
        if (tid == 0 && !kVecDecay) {
            Lam_s[len] = lnew;
            Lg[len] = lnew;
        }
        __syncthreads();  // the entry is in shared memory before the next token reads the log
    }
    if (tid == 0) st.log_len[unit] = len0 + T;
}

}  // namespace deltalog
