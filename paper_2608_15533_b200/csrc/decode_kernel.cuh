// Decode + append kernel: one CTA per (batch row, head).
//
// Per unit (Algorithm 1, append branch; Eq. 4 and Eq. 6):
//   lbar  = Lambda[len-1] (0 if the log is empty),  lbar' = lbar + lambda_t
//   delta ops:  y_k = S_base^T (e^{lbar'} . k) + sum_i ck_i U_i,   ck_i = sum_j k_j e^{lbar'_j - Lambda_ij} K_ij
//               y_q = S_base^T (e^{lbar'} . q) + sum_i cq_i U_i,   cq_i likewise with q
//               b   = beta (v - y_k);   out = scale (y_q + (q.k) b)
//   RWKV6:      y_r = S_base^T (e^{lbar} . r) + sum_i cr_i U_i  with the *old* lbar (pre-update readout)
//               b   = v;                out = y_r + (r . (bonus . k)) v
//   append:     K[len] = k, U[len] = b, Lambda[len] = lbar', len += 1.   S_base is never written.
//
// The base tile (4*d_k*d_v bytes, half of that for a bf16 base) is the only large read; it is requested
// first, as vector loads held in registers, before anything that depends on the (small) metadata.
#pragma once

#include "common.cuh"

namespace deltalog {

// Threads per CTA: 256 when a head dimension is 128; 128 at head size 64 x 64, where the tile is only
// 16 KiB and the run time of a CTA is one long latency chain (length -> snapshot and log -> coefficients):
// smaller CTAs let eight of them overlap their chains on an SM instead of four.  (The key dimension DK
// indexes the tile's rows, the value dimension DV its columns; they may differ.)
template <int DK, int DV>
__host__ __device__ constexpr int decode_threads() {
    return (DK >= 128 || DV >= 128) ? 256 : 128;
}

template <int DK, int DV, typename IO, typename UL>
__host__ __device__ constexpr size_t decode_smem_bytes(int op, int cap) {
    const size_t dl = (op == DELTALOG_GDN || op == DELTALOG_RETNET || op == DELTALOG_LINATTN) ? 1 : DK;
    size_t bytes = 0;
    bytes += sizeof(float) * DK * 4;                // q, k (raw), mul_k, mul_q
    bytes += sizeof(float) * DV;                    // b
    bytes += sizeof(float) * DK;                    // lbar_old (vector ops)
    bytes += sizeof(float) * 2 * kMaxCap;           // replay coefficients
    bytes += sizeof(float) * 2 * DV * (decode_threads<DK, DV>() / (DV / 4));  // cross-row-lane partial sums
    bytes += 16;                                    // scalars
    bytes += sizeof(UL) * (size_t)cap * DV;         // U log
    bytes += sizeof(IO) * (size_t)cap * DK;         // K log
    bytes += sizeof(float) * (((size_t)cap * dl + 3) / 4 * 4);  // Lambda log
    return bytes;
}

#ifndef DELTALOG_SIMPLE_CTAS
#define DELTALOG_SIMPLE_CTAS 2
#endif
template <int OP, int DK, int DV, typename IO, typename UL, typename BT = float>
__global__ void __launch_bounds__(decode_threads<DK, DV>(), decode_threads<DK, DV>() >= 256 ? DELTALOG_SIMPLE_CTAS : 8)
decode_append_kernel(StateArgs st, TokenArgs tk) {
    constexpr int NT = decode_threads<DK, DV>();
    constexpr int NW = NT / 32;
    constexpr bool kDelta = OpTraits<OP>::kDeltaRule;
    constexpr bool kPost = OpTraits<OP>::kPostReadout;
    constexpr bool kVecDecay = OpTraits<OP>::kVecDecay;
    constexpr int DL = kVecDecay ? DK : 1;
    constexpr int C4 = DV / 4;         // float4 columns per state row
    constexpr int RL = NT / C4;        // rows covered by one pass of the CTA
    constexpr int NP = DK / RL;        // passes over the tile
    constexpr int EPL = DK / 32;       // key elements per lane in a warp-wide dot product
    static_assert(NT >= DK && NT >= (kDelta ? 2 : 1) * DV, "one thread per key channel and per output column");

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.x / st.H, h = blockIdx.x % st.H;
    // Chained launch (see DELTALOG_HINT_BASE_UNTOUCHED): the slot list is read ahead of the preceding
    // kernel's completion only if there is none or the caller vouched for it (DELTALOG_HINT_SLOTS_STABLE).
    if (tk.slot_idx != nullptr && !(tk.hints & DELTALOG_HINT_SLOTS_STABLE)) asm volatile("griddepcontrol.wait;\n" ::: "memory");
    int slot;
    if (!resolve_slot(tk.slot_idx, b, st.num_slots, st.status, tid, slot)) return;
    const size_t unit = (size_t)slot * st.H + h;  // (slot, head) in the state pool
    const size_t row = (size_t)b * st.H + h;      // (batch row, head) in the token tensors
    const int cap = st.cap;

    // ---- 1. request the whole base tile (independent of every other load) -------------------
    const BT *Sg = static_cast<const BT *>(st.S_base) + unit * DK * DV;
    const int c4 = tid % C4, rl = tid / C4;
    float4 s[NP];
#pragma unroll
    for (int p = 0; p < NP; ++p) s[p] = base_ldg4<BT>(Sg + ((size_t)(p * RL + rl) * C4 + c4) * 4);

    // Programmatic dependent launch (see DELTALOG_HINT_BASE_UNTOUCHED): the kernel queued behind this
    // one may start as this one's CTAs retire; and if this kernel itself was started early, everything
    // the previous step wrote (lengths, log entries) is read only after that step has completed.  The
    // base tile above was requested before: the caller promised that the previous kernel leaves it alone.
    asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
    asm volatile("griddepcontrol.wait;\n" ::: "memory");
    const int len = st.log_len[unit];
    if (len >= cap || len < 0) {  // full: Algorithm 1's else-branch is the caller's job (deltalog_merge); < 0: corrupt
        if (tid == 0 && st.status) atomicOr(st.status, DELTALOG_STATUS_LOG_FULL);
        return;
    }

    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *q_s = reinterpret_cast<float *>(smem_raw);
    float *k_s = q_s + DK;
    float *mk_s = k_s + DK;     // e^{lbar'} . k
    float *mq_s = mk_s + DK;    // e^{lbar'} . q   (RWKV6: e^{lbar} . r)
    float *b_s = mq_s + DK;     // [DV] value-side factor, shared between the two output halves
    float *lold_s = b_s + DV;   // lbar (vector-decay ops)
    float *ck_s = lold_s + DK;  // [kMaxCap]
    float *cq_s = ck_s + kMaxCap;
    float *red_s = cq_s + kMaxCap;           // [RL][2][DV]
    float *scal_s = red_s + 2 * DV * RL;     // [0] = q.k  (or r.(bonus.k))
    UL *U_s = reinterpret_cast<UL *>(scal_s + 4);
    IO *K_s = reinterpret_cast<IO *>(U_s + (size_t)cap * DV);
    float *Lam_s = reinterpret_cast<float *>(K_s + (size_t)cap * DK);

    // ---- 2. stage the live log entries (asynchronously) and the token vectors ---------------
    const IO *Kg = static_cast<const IO *>(st.K_log) + unit * cap * DK;
    const UL *Ug = static_cast<const UL *>(st.U_log) + unit * cap * DV;
    const float *Lg = st.decay_log + unit * cap * DL;
    constexpr int kEntryBytes = DK * (int)sizeof(IO) + DV * (int)sizeof(UL) + DL * 4;
    const int total_units = tk.B * st.H;
    const uint64_t keep_rd = l2_policy_keep(st.keep_fraction(len, total_units, kEntryBytes));
    cta_cp_async_hint(K_s, Kg, len * DK * (int)sizeof(IO), tid, NT, keep_rd);
    cta_cp_async_hint(U_s, Ug, len * DV * (int)sizeof(UL), tid, NT, keep_rd);
    if (kVecDecay) cta_cp_async_hint(Lam_s, Lg, len * DK * (int)sizeof(float), tid, NT, keep_rd);
    cp_async_commit();
    if (!kVecDecay && tid < len) Lam_s[tid] = Lg[tid];

    const IO *qg = static_cast<const IO *>(tk.q) + tk.qk_row(b, h) * DK;
    const IO *kg = static_cast<const IO *>(tk.k) + tk.qk_row(b, h) * DK;
    const IO *vg = static_cast<const IO *>(tk.v) + row * DV;
    const float *gg = tk.g + row * DL;
    IO k_raw = from_f32<IO>(0.f);
    float lnew = 0.f;
    if (tid < DK) {
        const float qv = to_f32(qg[tid]);
        k_raw = kg[tid];
        const float kv = to_f32(k_raw);
        const float lold = (len > 0) ? Lg[(size_t)(len - 1) * DL + (kVecDecay ? tid : 0)] : 0.f;
        lnew = lold + (tk.g ? gg[kVecDecay ? tid : 0] : 0.f);  // no gate: plain linear attention
        q_s[tid] = qv;
        k_s[tid] = kv;
        lold_s[tid] = kPost ? lnew : lold;  // the decay level the replay coefficients refer to
        const float e = expf(kPost ? lnew : lold);
        mk_s[tid] = e * kv;
        mq_s[tid] = e * qv;
    }
    cp_async_wait_all();
    __syncthreads();

    // ---- 3. key-side replay coefficients: one warp per live entry ---------------------------
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
    if (warp == NW - 1) {  // q.k for the delta rule, r.(bonus.k) for RWKV6
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

    // ---- 4. base pass: two mat-vecs from one read of the tile -------------------------------
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

    // ---- 5. reduce, replay the value-side log, form b and the output, append ----------------
    const int which = tid / DV, c = tid % DV;  // which: 0 -> y_k half, 1 -> y_q half
    float y = 0.f;
    const bool active = kDelta ? (tid < 2 * DV) : (tid < DV);
    const int sel = kDelta ? which : 1;
    if (active) {
#pragma unroll
        for (int r = 0; r < RL; ++r) y += red_s[(r * 2 + sel) * DV + c];
        const float *coef = sel ? cq_s : ck_s;
        for (int i = 0; i < len; ++i) y = fmaf(coef[i], to_f32(U_s[i * DV + c]), y);
    }
    UL *Uout = static_cast<UL *>(st.U_log) + (unit * cap + len) * DV;
    IO *og = static_cast<IO *>(tk.out) + row * DV;
    // the new entry is read again by the following steps: same L2 policy as the log's reads
    const uint64_t keep_wr = l2_policy_keep(st.keep_fraction(len + 1, total_units, kEntryBytes));
    if (kDelta) {
        if (tid < DV) {
            const float bval = tk.beta[row] * (to_f32(vg[c]) - y);
            b_s[c] = bval;
            st_hint(Uout + c, from_f32<UL>(bval), keep_wr);
        }
        __syncthreads();
        if (active && which == 1) og[c] = from_f32<IO>(st.scale * fmaf(scal_s[0], b_s[c], y));
    } else if (active) {
        const IO v_raw = vg[c];
        og[c] = from_f32<IO>((kPost ? st.scale : 1.f) * fmaf(scal_s[0], to_f32(v_raw), y));
        st_hint(Uout + c, from_f32<UL>(to_f32(v_raw)), keep_wr);  // lossless: U log dtype equals the I/O dtype
    }
    if (tid < DK) {
        st_hint(static_cast<IO *>(st.K_log) + (unit * cap + len) * DK + tid, k_raw, keep_wr);
        if (kVecDecay) st_hint(st.decay_log + (unit * cap + len) * DL + tid, lnew, keep_wr);
    }
    if (tid == 0) {
        if (!kVecDecay) st_hint(st.decay_log + unit * cap + len, lnew, keep_wr);
        st.log_len[unit] = len + 1;
    }
}

}  // namespace deltalog
