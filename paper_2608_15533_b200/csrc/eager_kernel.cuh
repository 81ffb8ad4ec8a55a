// Eager dense comparator: one CTA per (batch row, head) reads the whole state tile (fp32, or bf16 and
// then rounded at every store, i.e. once per token) into registers, applies the token (Eq. 3 with the operator's factors from Table 1) and writes the
// whole tile back -- the per-token read-modify-write whose write half the log schedule removes.
//
//   delta ops:  S' = D(lambda) S;  b = beta (v - S'^T k);  S = S' + k b^T;
//               out = scale S^T q = scale (S'^T q + (q.k) b)
//   RWKV6:      out = S^T r + (r.(bonus.k)) v;  S = D(log w) S + k v^T
#pragma once

#include "common.cuh"

namespace deltalog {

template <int OP, int DK, int DV, typename IO, typename BT = float>
__global__ void __launch_bounds__(kThreads, 2)
eager_step_kernel(void *S, int32_t num_slots, int32_t H, float scale, int32_t *status, TokenArgs tk) {
    constexpr bool kDelta = OpTraits<OP>::kDeltaRule;
    constexpr bool kPost = OpTraits<OP>::kPostReadout;
    constexpr bool kVecDecay = OpTraits<OP>::kVecDecay;
    constexpr int DL = kVecDecay ? DK : 1;
    constexpr int C4 = DV / 4, RL = kThreads / C4, NP = DK / RL, EPL = DK / 32;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // (DELTALOG_HINT_WALK_DOWN: CTAs take the units from the last to the first -- alternated from step to step, a
    // step begins with the tiles the step before wrote last, which are still in L2)
    const int pair = (tk.hints & DELTALOG_HINT_WALK_DOWN) ? (int)gridDim.x - 1 - (int)blockIdx.x : (int)blockIdx.x;
    const int b = pair / H, h = pair % H;
    int slot;
    if (!resolve_slot(tk.slot_idx, b, num_slots, status, tid, slot)) return;
    const size_t unit = (size_t)slot * H + h, row = (size_t)b * H + h;

    BT *Sg = static_cast<BT *>(S) + unit * DK * DV;
    const int c4 = tid % C4, rl = tid / C4;
    float4 s[NP];
#pragma unroll
    for (int p = 0; p < NP; ++p) s[p] = base_load4<BT>(Sg + ((size_t)(p * RL + rl) * C4 + c4) * 4);

    __shared__ __align__(16) float q_s[DK], k_s[DK], a_s[DK], b_s[DV];
    __shared__ __align__(16) float red_s[2 * DV * RL];
    __shared__ float qk_s;

    const IO *vg = static_cast<const IO *>(tk.v) + row * DV;
    if (tid < DK) {
        q_s[tid] = to_f32(static_cast<const IO *>(tk.q)[tk.qk_row(b, h) * DK + tid]);
        k_s[tid] = to_f32(static_cast<const IO *>(tk.k)[tk.qk_row(b, h) * DK + tid]);
        a_s[tid] = tk.g ? expf(tk.g[row * DL + (kVecDecay ? tid : 0)]) : 1.f;  // no gate: plain linear attention
    }
    __syncthreads();
    if (warp == 0) {
        float d = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
            const int j = lane + 32 * e;
            const float w = kPost ? 1.f : tk.u_bonus[(size_t)h * DK + j];
            d = fmaf(q_s[j] * w, k_s[j], d);
        }
        d = warp_sum(d);
        if (lane == 0) qk_s = d;
    }

    float4 ak = make_float4(0.f, 0.f, 0.f, 0.f), aq = ak;
#pragma unroll
    for (int p = 0; p < NP; ++p) {
        const int r = p * RL + rl;
        if (kPost) {  // decay first; the readouts are taken on the decayed state
            const float a = a_s[r];
            s[p] = make_float4(a * s[p].x, a * s[p].y, a * s[p].z, a * s[p].w);
            if (kDelta) ak = fma4(k_s[r], s[p], ak);
        }
        aq = fma4(q_s[r], s[p], aq);  // RWKV6: readout on the old state
    }
    float4 *red4 = reinterpret_cast<float4 *>(red_s);
    if (kDelta) red4[(rl * 2 + 0) * C4 + c4] = ak;
    red4[(rl * 2 + 1) * C4 + c4] = aq;
    __syncthreads();

    const int which = tid / DV, c = tid % DV;
    const bool active = kDelta ? (tid < 2 * DV) : (tid < DV);
    const int sel = kDelta ? which : 1;
    float y = 0.f;
    if (active) {
#pragma unroll
        for (int r = 0; r < RL; ++r) y += red_s[(r * 2 + sel) * DV + c];
    }
    IO *og = static_cast<IO *>(tk.out) + row * DV;
    if (kDelta) {
        if (tid < DV) b_s[c] = tk.beta[row] * (to_f32(vg[c]) - y);
        __syncthreads();
        if (active && which == 1) og[c] = from_f32<IO>(scale * fmaf(qk_s, b_s[c], y));
    } else {
        if (active) {
            const float vv = to_f32(vg[c]);
            b_s[c] = vv;
            og[c] = from_f32<IO>((kPost ? scale : 1.f) * fmaf(qk_s, vv, y));
        }
        __syncthreads();
    }

    const float4 b4 = reinterpret_cast<const float4 *>(b_s)[c4];
#pragma unroll
    for (int p = 0; p < NP; ++p) {
        const int r = p * RL + rl;
        float4 x = s[p];
        if (!kPost) {
            const float a = a_s[r];
            x = make_float4(a * x.x, a * x.y, a * x.z, a * x.w);
        }
        base_store4<BT>(Sg + ((size_t)r * C4 + c4) * 4, fma4(k_s[r], b4, x));
    }
}

}  // namespace deltalog
