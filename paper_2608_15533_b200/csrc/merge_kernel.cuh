// Merge kernel: a CTA folds the live log of a (listed slot, head) unit into its dense base with a
// single read and a single write of the tile (Eq. 5 without the current-token term):
//
//   S_base[j, :] <- e^{lbar_j} S_base[j, :] + sum_{i<len} (e^{lbar_j - Lambda_ij} K_ij) U_i[:],   len <- 0
//
// with lbar = Lambda[len-1].  The key-side weights A_ij = e^{lbar_j - Lambda_ij} K_ij are formed
// once in shared memory; every thread then owns NP consecutive rows x 4 columns of the tile and
// applies the rank-len update to them in registers.
#pragma once

#include "common.cuh"

namespace deltalog {

// A [cap][DK], U [cap][DV] (fp32), e^{lbar} [DK]; then the log as it is stored, requested ahead of the length
// word: K [cap][DK] (I/O dtype), Lambda [cap][d_lambda] (fp32), and U [cap][DV] where it is not fp32 already.
template <int DK, int DV, typename IO, typename UL>
constexpr size_t merge_smem_bytes(int cap, bool vec_decay) {
    return sizeof(float) * ((size_t)cap * (DK + DV) + DK) + sizeof(IO) * (size_t)cap * DK +
           sizeof(float) * (((size_t)cap * (vec_decay ? DK : 1) + 3) / 4 * 4) +
           (sizeof(UL) == 4 ? 0 : sizeof(UL) * (size_t)cap * DV);
}

#ifndef DELTALOG_MERGE_PACK
#define DELTALOG_MERGE_PACK 16
#endif
constexpr int kMergePack = DELTALOG_MERGE_PACK;  // candidates per CTA of a predicate merge

#ifndef DELTALOG_MERGE_CTAS
#define DELTALOG_MERGE_CTAS 2
#endif
// PACK: (listed slot, head) pairs a CTA is responsible for: 1 when every listed unit is expected to
// fold, kMergePack (strided over the grid) for predicate merges over a batch with staggered fills, where most
// pairs are skipped.
template <int OP, int DK, int DV, typename IO, typename UL, int PACK, typename BT = float>
__global__ void __launch_bounds__(mat_threads<DK, DV>(), mat_threads<DK, DV>() <= 128 ? 2 * DELTALOG_MERGE_CTAS : DELTALOG_MERGE_CTAS)
merge_kernel(StateArgs st, const int32_t *slot_idx, int32_t only_if_full, int32_t n_pairs) {
    constexpr bool kVecDecay = OpTraits<OP>::kVecDecay;
    constexpr int DL = kVecDecay ? DK : 1;
    constexpr int NT = mat_threads<DK, DV>();
    constexpr int C4 = DV / 4, RL = NT / C4, NP = DK / RL;  // a thread owns NP consecutive rows x 4 columns

    const int tid = threadIdx.x;
    const int cap = st.cap;
    // The lengths of a CTA's PACK candidates are looked up in parallel first, so a CTA whose
    // candidates have nothing to fold costs one load latency, not PACK of them.
    __shared__ int s_unit[PACK], s_len[PACK];
    if (PACK > 1) {
        if (tid < PACK) {
            // candidates are strided over the grid: the heads of a full row are consecutive pairs, and
            // this way they land in different CTAs instead of queueing up in one
            const int pair = blockIdx.x + tid * gridDim.x;
            int len = 0, unit = 0;
            if (pair < n_pairs) {
                int slot;
                if (resolve_slot(slot_idx, pair / st.H, st.num_slots, st.status, 0, slot)) {
                    unit = slot * st.H + pair % st.H;
                    len = st.log_len[unit];
                    if (len <= 0 || len > cap || (only_if_full && len < cap)) len = 0;  // nothing to fold
                }
            }
            s_unit[tid] = unit;
            s_len[tid] = len;
        }
        __syncthreads();
    }
    for (int cand = 0; cand < PACK; ++cand) {
    int len;
    size_t unit;
    if (PACK > 1) {
        len = s_len[cand];
        if (len == 0) continue;
        unit = (size_t)s_unit[cand];
        if (cand > 0) __syncthreads();  // the previous candidate's shared-memory operands are no longer read
    } else {
        // CTAs take the pairs from the last to the first: the tiles written last (and still in L2 when the
        // kernel ends) are then the ones the next decode step, which walks upwards from pair 0, reads first
        const int pair = gridDim.x - 1 - blockIdx.x;
        int slot;
        if (!resolve_slot(slot_idx, pair / st.H, st.num_slots, st.status, tid, slot)) return;
        unit = (size_t)slot * st.H + pair % st.H;
        len = 0;  // read below, after the tile and the log have been requested
    }

    // each thread owns rows [rl*NP, rl*NP + NP) x columns [4*c4, 4*c4 + 4)
    BT *Sg = static_cast<BT *>(st.S_base) + unit * DK * DV;
    const int c4 = tid % C4, rl = tid / C4;
    float4 s[NP];
#pragma unroll
    for (int p = 0; p < NP; ++p) s[p] = base_load4<BT>(Sg + ((size_t)(rl * NP + p) * C4 + c4) * 4);

    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *A_s = reinterpret_cast<float *>(smem_raw);  // [len][DK]
    float *U_s = A_s + (size_t)cap * DK;               // [len][DV]
    float *e_s = U_s + (size_t)cap * DV;               // [DK]
    IO *K_raw = reinterpret_cast<IO *>(e_s + DK);      // [cap][DK] as stored
    float *L_raw = reinterpret_cast<float *>(K_raw + (size_t)cap * DK);  // [cap][DL]
    UL *U_raw = sizeof(UL) == 4 ? reinterpret_cast<UL *>(U_s) : reinterpret_cast<UL *>(L_raw + ((size_t)cap * DL + 3) / 4 * 4);

    const IO *Kg = static_cast<const IO *>(st.K_log) + unit * cap * DK;
    const UL *Ug = static_cast<const UL *>(st.U_log) + unit * cap * DV;
    const float *Lg = st.decay_log + unit * cap * DL;
    // Without the predicate every listed unit is expected to hold a full log: the whole log is requested
    // (asynchronously, into shared memory) together with the tile, BEFORE the length word is known -- a CTA's
    // run time is one chain of dependent memory round trips, and this takes one of them out.  Entries beyond
    // the live length are never used.  (Needs 16-byte aligned snapshot rows: cap % 4 == 0 for scalar decay.)
    const bool ahead = PACK == 1 && (kVecDecay || cap % 4 == 0);
    if (ahead) {
        cta_cp_async(K_raw, Kg, cap * DK * (int)sizeof(IO), tid, NT);
        cta_cp_async(U_raw, Ug, cap * DV * (int)sizeof(UL), tid, NT);
        cta_cp_async(L_raw, Lg, (cap * DL * 4 + 15) / 16 * 16, tid, NT);
        cp_async_commit();
    }
    if (PACK == 1) {
        len = st.log_len[unit];
        if (len <= 0 || len > cap || (only_if_full && len < cap)) {  // nothing to fold: no dense write
            cp_async_wait_all();
            return;
        }
    }
    if (ahead) {
        cp_async_wait_all();
        __syncthreads();
        const float *lbar_s = L_raw + (size_t)(len - 1) * DL;
        for (int x = tid * 4; x < len * DK; x += NT * 4) {
            const int i = x / DK, j = x % DK;
            float kv[4], w[4];
            load_vec<IO, 4>(K_raw + x, kv);
            if (kVecDecay) {
                const float4 lb = *reinterpret_cast<const float4 *>(lbar_s + j);
                const float4 li = *reinterpret_cast<const float4 *>(L_raw + (size_t)i * DK + j);
                w[0] = expf(lb.x - li.x), w[1] = expf(lb.y - li.y), w[2] = expf(lb.z - li.z), w[3] = expf(lb.w - li.w);
            } else {
                w[0] = w[1] = w[2] = w[3] = expf(lbar_s[0] - L_raw[i]);
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
        if (tid < DK) e_s[tid] = expf(lbar_s[kVecDecay ? tid : 0]);
    } else {
    const float *lbar = Lg + (size_t)(len - 1) * DL;
    // key-side weights A_ij = e^{lbar_j - Lambda_ij} K_ij and the value-side rows
    if (!kVecDecay) {  // one weight per entry: four elements per thread and pass
        for (int x = tid * 4; x < len * DK; x += NT * 4) {
            const float wi = expf(lbar[0] - Lg[x / DK]);
            float kv[4];
            load_vec<IO, 4>(Kg + x, kv);
            *reinterpret_cast<float4 *>(A_s + x) = make_float4(wi * kv[0], wi * kv[1], wi * kv[2], wi * kv[3]);
        }
        for (int x = tid * 4; x < len * DV; x += NT * 4) {
            float uv[4];
            load_vec<UL, 4>(Ug + x, uv);
            *reinterpret_cast<float4 *>(U_s + x) = make_float4(uv[0], uv[1], uv[2], uv[3]);
        }
    } else {  // one weight per element (measured: the element-wise loop is the faster one here)
        for (int x = tid; x < len * DK; x += NT) {
            const int i = x / DK, j = x % DK;
            A_s[x] = expf(lbar[j] - Lg[(size_t)i * DK + j]) * to_f32(Kg[x]);
        }
        for (int x = tid; x < len * DV; x += NT) U_s[x] = to_f32(Ug[x]);
    }
    if (tid < DK) e_s[tid] = expf(lbar[kVecDecay ? tid : 0]);
    }
    __syncthreads();

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
#pragma unroll
    for (int p = 0; p < NP; ++p) base_store4<BT>(Sg + ((size_t)(rl * NP + p) * C4 + c4) * 4, s[p]);
    if (tid == 0) st.log_len[unit] = 0;
    }
}

// Slot hand-over: empty the log of every head of the listed slots and, if given, install a new base.
template <typename BT = float>
__global__ void __launch_bounds__(kThreads) reset_slots_kernel(StateArgs st, const int32_t *slot_idx, const float *S_init,
                                                               int tile_elems /* d_k * d_v */) {
    const int i = blockIdx.x / st.H, h = blockIdx.x % st.H;
    int slot;
    if (!resolve_slot(slot_idx, i, st.num_slots, st.status, threadIdx.x, slot)) return;
    const size_t unit = (size_t)slot * st.H + h;
    if (S_init) {
        const float4 *src = reinterpret_cast<const float4 *>(S_init + ((size_t)i * st.H + h) * tile_elems);
        BT *dst = static_cast<BT *>(st.S_base) + unit * tile_elems;
        for (int x = threadIdx.x; x < tile_elems / 4; x += kThreads) base_store4<BT>(dst + 4 * x, src[x]);
    }
    if (threadIdx.x == 0) st.log_len[unit] = 0;
}

}  // namespace deltalog
