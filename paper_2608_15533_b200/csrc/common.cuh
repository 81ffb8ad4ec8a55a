// Shared device helpers for the DeltaLog kernels: dtype conversion, cp.async staging, warp sums.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "deltalog.h"

namespace deltalog {

constexpr int kThreads = 256;  // CTA size of the one-unit-per-CTA kernels at head size 128 (merge, fused step, eager)
constexpr int kWarps = kThreads / 32;
// CTA size of the materialisation kernels (merge, fused merge step): a thread holds D*D/NT elements of
// the tile in registers, so more threads mean fewer registers each and more resident warps.
#ifndef DELTALOG_MAT_THREADS
#define DELTALOG_MAT_THREADS 256
#endif
#ifndef DELTALOG_MAT_THREADS_64
#define DELTALOG_MAT_THREADS_64 128
#endif
template <int DK, int DV>
__host__ __device__ constexpr int mat_threads() {
    return (DK >= 128 && DV >= 128) ? DELTALOG_MAT_THREADS : (DK * DV <= 64 * 64 ? DELTALOG_MAT_THREADS_64 : 256);
}
constexpr int kMaxCap = 64;

// What the kernels need to know about an operator of Table 1.  The additive family shares kernels:
// plain linear attention runs the RetNet instantiation with a null gate pointer (lambda == 0).
template <int OP>
struct OpTraits {
    static constexpr bool kVecDecay = (OP == DELTALOG_KDA || OP == DELTALOG_RWKV6 || OP == DELTALOG_GLA);
    static constexpr bool kDeltaRule = (OP == DELTALOG_GDN || OP == DELTALOG_KDA);  // b = beta (v - S'^T k), else b = v
    static constexpr bool kPostReadout = (OP != DELTALOG_RWKV6);  // output read from S_t (scaled); RWKV6 reads S_{t-1}
    static constexpr bool kBonus = (OP == DELTALOG_RWKV6);
};

template <int DT> struct DType;
template <> struct DType<DELTALOG_F32> { using type = float; };
template <> struct DType<DELTALOG_BF16> { using type = __nv_bfloat16; };

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) {
    return __float2bfloat16_rn(x);
}

// Load N (2 or 4) consecutive elements as one vector access and widen them to fp32.
template <typename T, int N>
__device__ __forceinline__ void load_vec(const T *p, float (&out)[N]);
template <>
__device__ __forceinline__ void load_vec<float, 4>(const float *p, float (&out)[4]) {
    const float4 v = *reinterpret_cast<const float4 *>(p);
    out[0] = v.x, out[1] = v.y, out[2] = v.z, out[3] = v.w;
}
template <>
__device__ __forceinline__ void load_vec<float, 2>(const float *p, float (&out)[2]) {
    const float2 v = *reinterpret_cast<const float2 *>(p);
    out[0] = v.x, out[1] = v.y;
}
template <>
__device__ __forceinline__ void load_vec<__nv_bfloat16, 4>(const __nv_bfloat16 *p, float (&out)[4]) {
    const uint2 v = *reinterpret_cast<const uint2 *>(p);
    out[0] = __uint_as_float(v.x << 16), out[1] = __uint_as_float(v.x & 0xffff0000u);
    out[2] = __uint_as_float(v.y << 16), out[3] = __uint_as_float(v.y & 0xffff0000u);
}
template <>
__device__ __forceinline__ void load_vec<__nv_bfloat16, 2>(const __nv_bfloat16 *p, float (&out)[2]) {
    const uint32_t v = *reinterpret_cast<const uint32_t *>(p);
    out[0] = __uint_as_float(v << 16), out[1] = __uint_as_float(v & 0xffff0000u);
}

// Eight consecutive elements as 16-byte accesses, widened to fp32.
__device__ __forceinline__ void load8(const float *p, float (&out)[8]) {
    const float4 a = reinterpret_cast<const float4 *>(p)[0], b = reinterpret_cast<const float4 *>(p)[1];
    out[0] = a.x, out[1] = a.y, out[2] = a.z, out[3] = a.w, out[4] = b.x, out[5] = b.y, out[6] = b.z, out[7] = b.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16 *p, float (&out)[8]) {
    const uint4 v = *reinterpret_cast<const uint4 *>(p);
    out[0] = __uint_as_float(v.x << 16), out[1] = __uint_as_float(v.x & 0xffff0000u);
    out[2] = __uint_as_float(v.y << 16), out[3] = __uint_as_float(v.y & 0xffff0000u);
    out[4] = __uint_as_float(v.z << 16), out[5] = __uint_as_float(v.z & 0xffff0000u);
    out[6] = __uint_as_float(v.w << 16), out[7] = __uint_as_float(v.w & 0xffff0000u);
}

#ifndef DELTALOG_STREAM_BASE
#define DELTALOG_STREAM_BASE 1
#endif
// Four consecutive elements of a dense state tile as one vector access.  The state is fp32, or bf16
// (the 16-bit state of Section 2.2: half the bytes); arithmetic is fp32 either way, and a bf16 state is
// rounded to nearest even at the store -- the only place where precision is given up.
template <typename BT> __device__ __forceinline__ float4 base_load4(const BT *p);
template <> __device__ __forceinline__ float4 base_load4<float>(const float *p) {
    return *reinterpret_cast<const float4 *>(p);
}
template <> __device__ __forceinline__ float4 base_load4<__nv_bfloat16>(const __nv_bfloat16 *p) {
    const uint2 v = *reinterpret_cast<const uint2 *>(p);
    return make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xffff0000u), __uint_as_float(v.y << 16),
                       __uint_as_float(v.y & 0xffff0000u));
}
// The same as a streaming load (evict-first in L2): a decode step reads every base tile exactly once,
// hundreds of megabytes per launch, while the live log entries and the length words are read again by
// the next step -- marking the tiles as the first to go keeps the small, reused data in the 126 MB L2.
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;\n" : "=l"(p));
    return p;
}
// L2 policy for the live log, which every later step of the cycle reads again: last to be evicted -- but
// only for the fraction of its lines that L2 can hold.  A log that outgrows L2 is otherwise re-read
// cyclically and an LRU-like policy keeps none of it; with fraction = capacity / footprint a stable
// subset (chosen by the hardware from the address) stays resident and the rest streams.
#ifndef DELTALOG_L2_KEEP
#define DELTALOG_L2_KEEP 1
#endif
__device__ __forceinline__ uint64_t l2_policy_keep(float fraction) {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.L2::evict_first.b64 %0, %1;\n" : "=l"(p) : "f"(fraction));
    return p;
}
__device__ __forceinline__ void st_hint(float *p, float v, uint64_t policy) {
#if DELTALOG_L2_KEEP
    asm volatile("st.global.L2::cache_hint.f32 [%0], %1, %2;\n" ::"l"(p), "f"(v), "l"(policy) : "memory");
#else
    *p = v;
#endif
}
__device__ __forceinline__ void st_hint(__nv_bfloat16 *p, __nv_bfloat16 v, uint64_t policy) {
#if DELTALOG_L2_KEEP
    asm volatile("st.global.L2::cache_hint.b16 [%0], %1, %2;\n" ::"l"(p), "h"(__bfloat16_as_ushort(v)), "l"(policy) : "memory");
#else
    *p = v;
#endif
}
template <typename BT> __device__ __forceinline__ float4 base_ldg4(const BT *p);
template <> __device__ __forceinline__ float4 base_ldg4<float>(const float *p) {
#if DELTALOG_STREAM_BASE
    float4 v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.f32 {%0, %1, %2, %3}, [%4], %5;\n"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                 : "l"(p), "l"(l2_policy_evict_first()));
    return v;
#else
    return __ldg(reinterpret_cast<const float4 *>(p));
#endif
}
template <> __device__ __forceinline__ float4 base_ldg4<__nv_bfloat16>(const __nv_bfloat16 *p) {
#if DELTALOG_STREAM_BASE
    uint2 v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v2.u32 {%0, %1}, [%2], %3;\n"
                 : "=r"(v.x), "=r"(v.y)
                 : "l"(p), "l"(l2_policy_evict_first()));
#else
    const uint2 v = __ldg(reinterpret_cast<const uint2 *>(p));
#endif
    return make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xffff0000u), __uint_as_float(v.y << 16),
                       __uint_as_float(v.y & 0xffff0000u));
}
template <typename BT> __device__ __forceinline__ void base_store4(BT *p, const float4 &v);
template <> __device__ __forceinline__ void base_store4<float>(float *p, const float4 &v) {
    *reinterpret_cast<float4 *>(p) = v;
}
template <> __device__ __forceinline__ void base_store4<__nv_bfloat16>(__nv_bfloat16 *p, const float4 &v) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
    uint2 w;
    w.x = *reinterpret_cast<const uint32_t *>(&lo);
    w.y = *reinterpret_cast<const uint32_t *>(&hi);
    *reinterpret_cast<uint2 *>(p) = w;
}

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

__device__ __forceinline__ uint32_t smem_addr(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// Asynchronous 16-byte global -> shared copy (bypasses L1); both addresses 16-byte aligned.
__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gmem_src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(smem_addr(smem_dst)), "l"(gmem_src)
                 : "memory");
}
__device__ __forceinline__ void cp_async16_hint(void *smem_dst, const void *gmem_src, uint64_t policy) {
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;\n" ::"r"(smem_addr(smem_dst)), "l"(gmem_src),
                 "l"(policy)
                 : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;\n" ::: "memory"); }

// Cooperative async copy of `bytes` (multiple of 16) by the whole CTA of `nthreads` threads.
__device__ __forceinline__ void cta_cp_async(void *smem_dst, const void *gmem_src, int bytes, int tid,
                                             int nthreads = kThreads) {
    char *d = static_cast<char *>(smem_dst);
    const char *s = static_cast<const char *>(gmem_src);
    for (int off = tid * 16; off < bytes; off += nthreads * 16) cp_async16(d + off, s + off);
}

__device__ __forceinline__ void cta_cp_async_hint(void *smem_dst, const void *gmem_src, int bytes, int tid, int nthreads,
                                                  uint64_t policy) {
    char *d = static_cast<char *>(smem_dst);
    const char *s = static_cast<const char *>(gmem_src);
#if DELTALOG_L2_KEEP
    for (int off = tid * 16; off < bytes; off += nthreads * 16) cp_async16_hint(d + off, s + off, policy);
#else
    for (int off = tid * 16; off < bytes; off += nthreads * 16) cp_async16(d + off, s + off);
#endif
}

__device__ __forceinline__ float4 fma4(float a, const float4 &x, const float4 &acc) {
    return make_float4(fmaf(a, x.x, acc.x), fmaf(a, x.y, acc.y), fmaf(a, x.z, acc.z), fmaf(a, x.w, acc.w));
}

// Rank-len update of a thread's NP consecutive rows x 4 columns held in registers:
//     s[p] += sum_{i<len} A_i[p] * u_i,   load_a(i, p4) -> A_i for rows 4*p4 .. 4*p4+3,  load_u(i) -> u_i.
// The accumulators are kept as pairs of rows so that one packed fp32 FMA (two lanes per instruction)
// serves two rows: per entry 4 register packs and NP*2 packed FMAs instead of NP*4 scalar ones.
// Every element sees the same fused multiply-adds in the same order as the scalar form.
#ifndef DELTALOG_FFMA2
#define DELTALOG_FFMA2 1
#endif
template <int NP, typename LoadA, typename LoadU>
__device__ __forceinline__ void rank_update(float4 (&s)[NP], int len, LoadA load_a, LoadU load_u) {
    static_assert(NP % 4 == 0, "rows come in groups of four");
#if DELTALOG_FFMA2
    float2 acc[NP / 2][4];
#pragma unroll
    for (int pp = 0; pp < NP / 2; ++pp) {
        acc[pp][0] = make_float2(s[2 * pp].x, s[2 * pp + 1].x);
        acc[pp][1] = make_float2(s[2 * pp].y, s[2 * pp + 1].y);
        acc[pp][2] = make_float2(s[2 * pp].z, s[2 * pp + 1].z);
        acc[pp][3] = make_float2(s[2 * pp].w, s[2 * pp + 1].w);
    }
    for (int i = 0; i < len; ++i) {
        const float4 u = load_u(i);
        const float2 u0 = make_float2(u.x, u.x), u1 = make_float2(u.y, u.y);
        const float2 u2 = make_float2(u.z, u.z), u3 = make_float2(u.w, u.w);
#pragma unroll
        for (int p4 = 0; p4 < NP / 4; ++p4) {
            const float4 a = load_a(i, p4);
            const float2 a01 = make_float2(a.x, a.y), a23 = make_float2(a.z, a.w);
            acc[2 * p4][0] = __ffma2_rn(a01, u0, acc[2 * p4][0]);
            acc[2 * p4][1] = __ffma2_rn(a01, u1, acc[2 * p4][1]);
            acc[2 * p4][2] = __ffma2_rn(a01, u2, acc[2 * p4][2]);
            acc[2 * p4][3] = __ffma2_rn(a01, u3, acc[2 * p4][3]);
            acc[2 * p4 + 1][0] = __ffma2_rn(a23, u0, acc[2 * p4 + 1][0]);
            acc[2 * p4 + 1][1] = __ffma2_rn(a23, u1, acc[2 * p4 + 1][1]);
            acc[2 * p4 + 1][2] = __ffma2_rn(a23, u2, acc[2 * p4 + 1][2]);
            acc[2 * p4 + 1][3] = __ffma2_rn(a23, u3, acc[2 * p4 + 1][3]);
        }
    }
#pragma unroll
    for (int pp = 0; pp < NP / 2; ++pp) {
        s[2 * pp] = make_float4(acc[pp][0].x, acc[pp][1].x, acc[pp][2].x, acc[pp][3].x);
        s[2 * pp + 1] = make_float4(acc[pp][0].y, acc[pp][1].y, acc[pp][2].y, acc[pp][3].y);
    }
#else
    for (int i = 0; i < len; ++i) {
        const float4 u = load_u(i);
#pragma unroll
        for (int p4 = 0; p4 < NP / 4; ++p4) {
            const float4 a = load_a(i, p4);
            s[4 * p4 + 0] = fma4(a.x, u, s[4 * p4 + 0]);
            s[4 * p4 + 1] = fma4(a.y, u, s[4 * p4 + 1]);
            s[4 * p4 + 2] = fma4(a.z, u, s[4 * p4 + 2]);
            s[4 * p4 + 3] = fma4(a.w, u, s[4 * p4 + 3]);
        }
    }
#endif
}

// The same update with one scalar FMA per element (identical results: every element sees the same fused
// multiply-adds in the same order).  Two resident CTAs that stay on an SM for the whole launch share the
// packed-FMA pipe badly -- the older CTA's warps are served first and the younger one's rank update takes
// three times as long (measured) -- while scalar FMAs are shared evenly.
template <int NP, typename LoadA, typename LoadU>
__device__ __forceinline__ void rank_update_scalar(float4 (&s)[NP], int len, LoadA load_a, LoadU load_u) {
    static_assert(NP % 4 == 0, "rows come in groups of four");
    for (int i = 0; i < len; ++i) {
        const float4 u = load_u(i);
#pragma unroll
        for (int p4 = 0; p4 < NP / 4; ++p4) {
            const float4 a = load_a(i, p4);
            s[4 * p4 + 0] = fma4(a.x, u, s[4 * p4 + 0]);
            s[4 * p4 + 1] = fma4(a.y, u, s[4 * p4 + 1]);
            s[4 * p4 + 2] = fma4(a.z, u, s[4 * p4 + 2]);
            s[4 * p4 + 3] = fma4(a.w, u, s[4 * p4 + 3]);
        }
    }
}

// Resolve the pool slot of batch row b; returns false when the row must be skipped.
__device__ __forceinline__ bool resolve_slot(const int32_t *slot_idx, int b, int num_slots, int32_t *status,
                                             int tid, int &slot) {
    slot = slot_idx ? slot_idx[b] : b;
    if (slot < 0) return false;  // padding row
    if (slot >= num_slots) {
        if (tid == 0 && status) atomicOr(status, DELTALOG_STATUS_BAD_SLOT);
        return false;
    }
    return true;
}

// Token-side arguments shared by the decode and eager kernels.
struct TokenArgs {
    const void *q, *k, *v;
    const float *g, *beta, *u_bonus;
    const int32_t *slot_idx;
    void *out;
    int32_t B;
    int32_t H_qk;      // query/key heads
    int32_t qk_group;  // state heads per query/key head (H / H_qk)
    int32_t hints;     // DELTALOG_HINT_* bits of the descriptor
    // row of q / k that (batch row b, state head h) reads
    __device__ __forceinline__ size_t qk_row(int b, int h) const { return (size_t)b * H_qk + h / qk_group; }
};

struct StateArgs {
    void *S_base;  // fp32 or bf16 tiles (the kernels' BT template parameter)
    void *K_log, *U_log;
    float *decay_log;
    int32_t *log_len;
    int32_t *status;
    int32_t num_slots, H, cap;
    float scale;
    float l2_keep_bytes;  // how much of the live log L2 is asked to hold on to (see l2_policy_keep)
    float l2_pin_bytes;   // how much of the dense base L2 is asked to hold on to across steps
    // fraction of a unit's log lines to keep, when every unit of this launch holds about len + 1 entries
    __device__ __forceinline__ float keep_fraction(int len, int total_units, int entry_bytes) const {
        // (never zero: the policy instruction wants a fraction in (0, 1])
        return fminf(1.f, fmaxf(1e-3f, l2_keep_bytes / ((float)total_units * (float)(len + 1) * (float)entry_bytes)));
    }
};

}  // namespace deltalog
