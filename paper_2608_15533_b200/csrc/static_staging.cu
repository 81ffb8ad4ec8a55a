// deltalog_decode_step_host_static: the host-buffer decode step without any caller-provided
// staging memory.  The device-side staging area that deltalog_decode_step_host takes from the
// caller lives here in a fixed-size static __device__ array instead, so this entry point makes no
// allocation of any kind.  See include/deltalog.h for the contract.
#include <cstdint>
#include <mutex>

#include <cuda_runtime.h>

#include "deltalog.h"
#include "validate.h"

namespace {

// The staging area.  Every GPU that loads this library carries it until the process exits.
static __device__ __align__(256) unsigned char g_static_staging[DELTALOG_STATIC_STAGING_BYTES];

// In host code `g_static_staging` is only a handle for the runtime, not a device address; the
// address is looked up once per device (with that device current) and cached here.
constexpr int kMaxDevices = 64;
void *g_staging_addr[kMaxDevices] = {};
std::mutex g_staging_mutex;

int staging_address(void **out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return DELTALOG_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_staging_mutex);
    if (!g_staging_addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_staging) != cudaSuccess || !p) return DELTALOG_ERR_CUDA;
        g_staging_addr[dev] = p;
    }
    *out = g_staging_addr[dev];
    return DELTALOG_OK;
}

size_t round256(size_t x) { return (x + 255) / 256 * 256; }

}  // namespace

extern "C" int deltalog_decode_step_host_static(const deltalog_desc *desc, const deltalog_state *state,
                                                const void *host_q, const void *host_k, const void *host_v,
                                                const float *host_g, const float *host_beta,
                                                const float *u_bonus, const int32_t *slot_idx, int32_t B,
                                                void *host_out, void *stream) {
    // Every argument check of the step runs here, before anything touches the shared array or the
    // stream: a call that is going to be rejected must not clobber what an earlier call staged.
    if (!desc || B < 0 || desc->H <= 0 || desc->d_k <= 0 || desc->d_v <= 0) return DELTALOG_ERR_INVALID_ARG;
    if (desc->io_dtype != DELTALOG_F32 && desc->io_dtype != DELTALOG_BF16) return DELTALOG_ERR_INVALID_ARG;
    if (int rc = deltalog::validate_desc(desc)) return rc;
    if (!host_q || !host_k || !host_v || !host_out) return DELTALOG_ERR_INVALID_ARG;
    if (deltalog::op_has_gate(desc->op) && !host_g) return DELTALOG_ERR_INVALID_ARG;
    if (deltalog::op_delta_rule(desc->op) && !host_beta) return DELTALOG_ERR_INVALID_ARG;
    if (desc->op == DELTALOG_RWKV6 && !u_bonus) return DELTALOG_ERR_INVALID_ARG;
    if (B == 0) return DELTALOG_OK;

    // carve q | k | v | g | beta | out out of the static area, 256-byte aligned each
    const size_t units = (size_t)B * (size_t)desc->H;
    const size_t esz = desc->io_dtype == DELTALOG_F32 ? 4 : 2;
    const size_t qk_heads = desc->H_qk > 0 ? (size_t)desc->H_qk : (size_t)desc->H;  // grouped heads: q, k are [B, H_qk, d_k]
    const size_t qk = round256((size_t)B * qk_heads * (size_t)desc->d_k * esz);
    const size_t vo = round256(units * (size_t)desc->d_v * esz);
    const size_t gb = round256(units * (size_t)(desc->op == DELTALOG_KDA || desc->op == DELTALOG_RWKV6 || desc->op == DELTALOG_GLA ? desc->d_k : 1) * sizeof(float));
    const size_t bb = round256(units * sizeof(float));
    if (2 * qk + 2 * vo + gb + bb > (size_t)DELTALOG_STATIC_STAGING_BYTES) return DELTALOG_ERR_STATIC_LIMIT;

    if (int rc = deltalog::validate_state(state)) return rc;

    void *base = nullptr;
    if (int rc = staging_address(&base)) return rc;
    unsigned char *p = static_cast<unsigned char *>(base);
    deltalog_staging stg;
    stg.q = p;
    stg.k = p + qk;
    stg.v = p + 2 * qk;
    stg.g = reinterpret_cast<float *>(p + 2 * qk + vo);
    stg.beta = reinterpret_cast<float *>(p + 2 * qk + vo + gb);
    stg.out = p + 2 * qk + vo + gb + bb;
    stg.packed = 0;  // nothing is known about the caller's host buffers
    // The area keeps whatever the previous call left behind.  Rows the kernel skips (padding, bad
    // slot, full log) are not written, so the output region is cleared first: those rows read back
    // as zeros instead of as the previous call's output.
    if (cudaMemsetAsync(stg.out, 0, vo, static_cast<cudaStream_t>(stream)) != cudaSuccess) return DELTALOG_ERR_CUDA;
    return deltalog_decode_step_host(desc, state, &stg, host_q, host_k, host_v, host_g, host_beta, u_bonus,
                                     slot_idx, B, host_out, stream);
}
