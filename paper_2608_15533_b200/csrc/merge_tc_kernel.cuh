// Tensor-core merge (head size 128): the rank-len update of Eq. 5,
//
//   S_base[j, :] <- e^{lbar_j} S_base[j, :] + sum_{i<len} (e^{lbar_j - Lambda_ij} K_ij) U_i[:],   len <- 0,
//
// with the contraction over the log entries on the 5th-generation tensor cores: one CTA per unit
// forms the 128 x 128 x len product A^T U with tcgen05.mma (kind::tf32, operands in shared memory,
// fp32 accumulator in tensor memory) and adds it to the decayed base tile on the way out.
//
// fp32 accuracy from tf32 inputs: every operand x is split as x = hi + lo with hi the leading 11
// bits of the significand (exactly representable in tf32) and lo = x - hi (exact in fp32), and the
// product is accumulated as hi*hi + lo*hi + hi*lo (the dropped lo*lo term is 2^-22 relative).
//
// Operand layout (K-major, no swizzle): per step of K = 8 entries, element (row r, entry k) of an
// operand sits at ((k % 8) / 4) * 2048 + (r / 8) * 128 + (r % 8) * 16 + (k % 4) * 4 bytes: 8-row x
// 16-byte core matrices, leading (K) byte offset 2048, stride (row-group) byte offset 128.
//
// The base tile is read and written in the register layout of the tensor-memory load
// (tcgen05.ld.16x256b): a warp instruction touches 8 rows x 32 contiguous bytes, i.e. whole sectors.
#pragma once

#include "common.cuh"
#include "decode_pipelined.cuh"  // mbarrier helpers, bounded_wait

namespace deltalog {

constexpr int kTcD = 128;
constexpr int kTcOperandBytes = 4096;  // one operand, one K = 8 step: 128 rows x 8 entries x 4 B

__host__ __device__ constexpr int tc_ksteps(int cap) { return (cap + 7) / 8; }
// A_hi, A_lo, U_hi, U_lo for every step, the row scales, barrier + tensor-memory slot + abort flag
template <int OP, typename IO, typename UL>
__host__ __device__ constexpr size_t merge_tc_smem_bytes(int cap) {
    return (size_t)4 * kTcOperandBytes * tc_ksteps(cap) + kTcD * sizeof(float) + 64 +        // operands, e, misc
           sizeof(float) * (OpTraits<OP>::kVecDecay ? (size_t)cap * kTcD : kMaxCap) +         // Lambda / weights
           (sizeof(UL) + sizeof(IO)) * (size_t)cap * kTcD;                                     // raw U, raw K
}

__device__ __forceinline__ int tc_operand_offset(int r, int k) {
    return (k / 8) * (4 * kTcOperandBytes) + ((k % 8) / 4) * 2048 + (r / 8) * 128 + (r % 8) * 16 + (k % 4) * 4;
}

// Shared-memory matrix descriptor: start address, leading and stride byte offsets (all / 16), version 1.
__device__ __forceinline__ uint64_t tc_smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | ((uint64_t)1 << 46);
}

// D[tmem] (+)= A * B^T for one K = 8 step, M = N = 128, tf32 inputs, fp32 accumulation.
__device__ __forceinline__ void tc_mma_tf32(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, bool accumulate) {
    // instruction descriptor: D f32, A and B tf32, both K-major, N = 128, M = 128
    constexpr uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
        " tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n}\n" ::"r"(tmem_d),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate ? 1u : 0u), "r"(0), "r"(0), "r"(0), "r"(0)
        : "memory");
}

__device__ __forceinline__ void tc_split(float x, float &hi, float &lo) {
    hi = __uint_as_float(__float_as_uint(x) & 0xffffe000u);
    lo = x - hi;
}

// 16 lanes x 256 bits, 8 repetitions along the columns: thread t receives, for column block cb,
// r[4cb+0..1] = (lane t/4, columns 8cb + 2(t%4) + {0,1}) and r[4cb+2..3] = the same columns of lane t/4 + 8.
__device__ __forceinline__ void tc_load_16x256b_x8(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.16x256b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
}

template <int OP, typename IO, typename UL>
__global__ void __launch_bounds__(kThreads, 2)
merge_tc_kernel(StateArgs st, const int32_t *slot_idx, int32_t only_if_full) {
    constexpr int D = kTcD;
    constexpr bool kVecDecay = OpTraits<OP>::kVecDecay;
    constexpr int DL = kVecDecay ? D : 1;
    constexpr int kTmemCols = 128;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cap = st.cap;
    const int pair = blockIdx.x;
    int slot;
    if (!resolve_slot(slot_idx, pair / st.H, st.num_slots, st.status, tid, slot)) return;
    const size_t unit = (size_t)slot * st.H + pair % st.H;
    const int len = st.log_len[unit];
    if (len <= 0 || len > cap || (only_if_full && len < cap)) return;  // nothing to fold: no dense write
    const int ksteps = (len + 7) / 8;

    extern __shared__ __align__(16) unsigned char smem_raw[];
    unsigned char *ops = smem_raw;  // per step: A_hi | A_lo | U_hi | U_lo, 4 KiB each
    float *e_s = reinterpret_cast<float *>(smem_raw + (size_t)4 * kTcOperandBytes * tc_ksteps(cap));
    uint64_t *bar = reinterpret_cast<uint64_t *>(e_s + D);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bar + 1);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    // raw copies of the live entries: Lambda (vector decay) or the entry weights (scalar decay), U, K
    float *L_raw = reinterpret_cast<float *>(smem_raw + (size_t)4 * kTcOperandBytes * tc_ksteps(cap) + D * sizeof(float) + 64);
    UL *U_raw = reinterpret_cast<UL *>(L_raw + (kVecDecay ? (size_t)cap * D : kMaxCap));
    IO *K_raw = reinterpret_cast<IO *>(U_raw + (size_t)cap * D);

    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_addr(tmem_slot)),
                     "r"(kTmemCols));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::);
    }
    if (tid == 0) {
        mbar_init(smem_addr(bar), 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }

    // ---- the base tile, in the register layout of the tensor-memory load -------------------------
    // warp w: lane quarter q = w % 4 (rows 32q .. 32q+31), column half w / 4; per 16-row half hh and
    // 8-column block cb a thread holds rows 32q + 16hh + lane/4 (+8), columns 64 half + 8cb + 2(lane%4) + {0,1}
    const int q = warp & 3, half = warp >> 2;
    float *Sg = static_cast<float *>(st.S_base) + unit * D * D;  // fp32 base only
    const int row_base = 32 * q + lane / 4, col_base = 64 * half + 2 * (lane % 4);
    float2 s[2][8][2];
#pragma unroll
    for (int hh = 0; hh < 2; ++hh)
#pragma unroll
        for (int cb = 0; cb < 8; ++cb) {
            const float *p = Sg + (size_t)(row_base + 16 * hh) * D + col_base + 8 * cb;
            s[hh][cb][0] = *reinterpret_cast<const float2 *>(p);
            s[hh][cb][1] = *reinterpret_cast<const float2 *>(p + 8 * D);
        }

    // ---- raw log entries into shared memory (asynchronously), entry weights for scalar decay -----
    const IO *Kg = static_cast<const IO *>(st.K_log) + unit * cap * D;
    const UL *Ug = static_cast<const UL *>(st.U_log) + unit * cap * D;
    const float *Lg = st.decay_log + unit * cap * DL;
    const float *lbar = Lg + (size_t)(len - 1) * DL;
    cta_cp_async(K_raw, Kg, len * D * (int)sizeof(IO), tid);
    cta_cp_async(U_raw, Ug, len * D * (int)sizeof(UL), tid);
    if (kVecDecay) cta_cp_async(L_raw, Lg, len * D * (int)sizeof(float), tid);
    cp_async_commit();
    if (!kVecDecay && tid < len) L_raw[tid] = expf(lbar[0] - Lg[tid]);  // w_i = e^{lbar - Lambda_i}
    cp_async_wait_all();
    __syncthreads();

    // ---- operands: A[j][i] = e^{lbar_j - Lambda_ij} K_ij and B[c][i] = U_i[c], split hi / lo ------
    for (int it = tid; it < D * 2 * ksteps; it += kThreads) {
        const int r = it % D, kc = it / D;  // row (key channel j / value column c) and group of four entries
        float ah[4], al[4], uh[4], ul[4];
        const float lb = kVecDecay ? L_raw[(size_t)(len - 1) * D + r] : 0.f;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int i = 4 * kc + e;
            float a = 0.f, u = 0.f;  // entries past the live length contribute nothing
            if (i < len) {
                const float w = kVecDecay ? expf(lb - L_raw[(size_t)i * D + r]) : L_raw[i];
                a = w * to_f32(K_raw[(size_t)i * D + r]);
                u = to_f32(U_raw[(size_t)i * D + r]);
            }
            tc_split(a, ah[e], al[e]);
            tc_split(u, uh[e], ul[e]);
        }
        unsigned char *dst = ops + tc_operand_offset(r, 4 * kc);
        *reinterpret_cast<float4 *>(dst) = make_float4(ah[0], ah[1], ah[2], ah[3]);
        *reinterpret_cast<float4 *>(dst + kTcOperandBytes) = make_float4(al[0], al[1], al[2], al[3]);
        *reinterpret_cast<float4 *>(dst + 2 * kTcOperandBytes) = make_float4(uh[0], uh[1], uh[2], uh[3]);
        *reinterpret_cast<float4 *>(dst + 3 * kTcOperandBytes) = make_float4(ul[0], ul[1], ul[2], ul[3]);
    }
    if (tid < D) e_s[tid] = expf(kVecDecay ? L_raw[(size_t)(len - 1) * D + tid] : lbar[0]);
    asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");  // generic writes -> tensor-core reads
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    const uint32_t tmem = *tmem_slot;

    // ---- the contraction: three tf32 products per step, issued by one thread ----------------------
    if (tid == 0) {
        bool first = true;
        for (int sidx = 0; sidx < ksteps; ++sidx) {
            const uint32_t base = smem_addr(ops + (size_t)sidx * 4 * kTcOperandBytes);
            const uint64_t a_hi = tc_smem_desc(base, 2048, 128), a_lo = tc_smem_desc(base + kTcOperandBytes, 2048, 128);
            const uint64_t u_hi = tc_smem_desc(base + 2 * kTcOperandBytes, 2048, 128);
            const uint64_t u_lo = tc_smem_desc(base + 3 * kTcOperandBytes, 2048, 128);
            tc_mma_tf32(tmem, a_hi, u_hi, !first);
            tc_mma_tf32(tmem, a_lo, u_hi, true);
            tc_mma_tf32(tmem, a_hi, u_lo, true);
            first = false;
        }
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(smem_addr(bar))
                     : "memory");
    }
    const bool done = bounded_wait(smem_addr(bar), 0u, abort_flag);
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");

    // ---- S <- e^{lbar} S + A^T U, straight from tensor memory into the registers that hold the tile --
    if (done) {
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            uint32_t acc[32];
            tc_load_16x256b_x8(tmem + ((uint32_t)(32 * q + 16 * hh) << 16) + 64 * half, acc);
            const float e0 = e_s[row_base + 16 * hh], e1 = e_s[row_base + 16 * hh + 8];
#pragma unroll
            for (int cb = 0; cb < 8; ++cb) {
                float *p = Sg + (size_t)(row_base + 16 * hh) * D + col_base + 8 * cb;
                *reinterpret_cast<float2 *>(p) =
                    make_float2(fmaf(e0, s[hh][cb][0].x, __uint_as_float(acc[4 * cb + 0])),
                                fmaf(e0, s[hh][cb][0].y, __uint_as_float(acc[4 * cb + 1])));
                *reinterpret_cast<float2 *>(p + 8 * D) =
                    make_float2(fmaf(e1, s[hh][cb][1].x, __uint_as_float(acc[4 * cb + 2])),
                                fmaf(e1, s[hh][cb][1].y, __uint_as_float(acc[4 * cb + 3])));
            }
        }
        if (tid == 0) st.log_len[unit] = 0;
    } else if (tid == 0 && st.status) {
        atomicOr(st.status, DELTALOG_STATUS_TIMEOUT);
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(kTmemCols));
}

}  // namespace deltalog
