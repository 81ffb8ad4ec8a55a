// C ABI of the DeltaLog decode library: host-side argument validation; the kernels are chosen and
// launched by the dispatch functions of the launch_*.cu translation units.
// Declarations and the contract of every entry point are in include/deltalog.h.
#include "launch_common.cuh"

namespace deltalog {

std::atomic<uint64_t> g_launches{0};

namespace {

int qk_heads(const deltalog_desc *d) { return d->H_qk > 0 ? d->H_qk : d->H; }

TokenArgs make_token_args(const deltalog_desc *d, const void *q, const void *k, const void *v, const float *g,
                          const float *beta, const float *u_bonus, const int32_t *slot_idx, void *out, int32_t B) {
    // plain linear attention has no gate: the kernels see a null pointer and use lambda = 0
    return TokenArgs{q, k, v, op_has_gate(d->op) ? g : nullptr, beta, u_bonus, slot_idx, out, B, qk_heads(d), d->H / qk_heads(d),
                     d->hints};
}

size_t round256(size_t x) { return (x + 255) / 256 * 256; }

// Host and staging buffers are "packed" when q, k, v, g (if the operator has a gate) and beta (delta
// rule) follow one another in this order, each starting on the next 256-byte boundary after the
// previous one ends, on BOTH sides: the five copies then collapse into one over the whole block.
// Returns the block's size, or 0 when the layout is not packed.
size_t packed_block_bytes(const deltalog_desc *d, const deltalog_staging *stg, const void *hq, const void *hk,
                          const void *hv, const float *hg, const float *hbeta, size_t qk_vec, size_t vec,
                          size_t gbytes, size_t units) {
    if (!stg->packed) return 0;  // adjacency alone proves nothing: the block must be one allocation
    const char *h = static_cast<const char *>(hq);
    const char *s = static_cast<const char *>(stg->q);
    size_t off = round256(qk_vec);
    if (static_cast<const char *>(hk) != h + off || static_cast<const char *>(stg->k) != s + off) return 0;
    off += round256(qk_vec);
    if (static_cast<const char *>(hv) != h + off || static_cast<const char *>(stg->v) != s + off) return 0;
    size_t end = off + vec;
    off += round256(vec);
    if (op_has_gate(d->op)) {
        if (reinterpret_cast<const char *>(hg) != h + off || reinterpret_cast<const char *>(stg->g) != s + off) return 0;
        end = off + gbytes;
        off += round256(gbytes);
    }
    if (op_delta_rule(d->op)) {
        if (reinterpret_cast<const char *>(hbeta) != h + off || reinterpret_cast<const char *>(stg->beta) != s + off) return 0;
        end = off + units * sizeof(float);
    }
    return end;
}

StateArgs make_state_args(const deltalog_desc *d, const deltalog_state *s) {
    StateArgs a;
    a.S_base = s->S_base;
    a.K_log = s->K_log;
    a.U_log = s->U_log;
    a.decay_log = s->decay_log;
    a.log_len = s->log_len;
    a.status = s->status;
    a.num_slots = d->num_slots;
    a.H = d->H;
    a.cap = d->cap;
    a.scale = d->scale;
    static const int keep_mb = env_int("DELTALOG_L2_KEEP_MB", 40);
    a.l2_keep_bytes = (float)keep_mb * 1048576.f;
    a.l2_pin_bytes = 0.f;  // set per launch by the pipelined decode kernel's launcher
    return a;
}


}  // namespace
}  // namespace deltalog

using namespace deltalog;

extern "C" {

int deltalog_decode_step(const deltalog_desc *desc, const deltalog_state *state, const void *q,
                         const void *k, const void *v, const float *g, const float *beta,
                         const float *u_bonus, const int32_t *slot_idx, int32_t B, void *out,
                         void *stream) {
    if (int rc = validate_desc(desc)) return rc;
    if (int rc = validate_state(state)) return rc;
    if (int rc = validate_token(desc, q, k, v, g, beta, u_bonus, B, out)) return rc;
    if (B == 0) return DELTALOG_OK;
    const StateArgs st = make_state_args(desc, state);
    const TokenArgs tk = make_token_args(desc, q, k, v, g, beta, u_bonus, slot_idx, out, B);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    return (desc->d_k == 128 && desc->d_v == 128) ? dispatch_decode_128(desc, st, tk, s) : dispatch_decode_other(desc, st, tk, s);
}

int deltalog_decode_steps(const deltalog_desc *desc, const deltalog_state *state, const void *q, const void *k,
                          const void *v, const float *g, const float *beta, const float *u_bonus,
                          const int32_t *slot_idx, int32_t B, int32_t T, void *out, void *stream) {
    if (int rc = validate_desc(desc)) return rc;
    if (int rc = validate_state(state)) return rc;
    if (int rc = validate_token(desc, q, k, v, g, beta, u_bonus, B, out)) return rc;
    if (T < 1 || T > desc->cap) return DELTALOG_ERR_CAP_RANGE;
    if (B == 0) return DELTALOG_OK;
    const StateArgs st = make_state_args(desc, state);
    const TokenArgs tk = make_token_args(desc, q, k, v, g, beta, u_bonus, slot_idx, out, B);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    return dispatch_decode_multi(desc, st, tk, T, s);
}

int deltalog_decode_merge_step(const deltalog_desc *desc, const deltalog_state *state, const void *q,
                               const void *k, const void *v, const float *g, const float *beta,
                               const float *u_bonus, const int32_t *slot_idx, int32_t B, void *out,
                               void *stream) {
    if (int rc = validate_desc(desc)) return rc;
    if (int rc = validate_state(state)) return rc;
    if (int rc = validate_token(desc, q, k, v, g, beta, u_bonus, B, out)) return rc;
    if (B == 0) return DELTALOG_OK;
    const StateArgs st = make_state_args(desc, state);
    const TokenArgs tk = make_token_args(desc, q, k, v, g, beta, u_bonus, slot_idx, out, B);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    return dispatch_fused_step(desc, st, tk, s);
}

int deltalog_merge(const deltalog_desc *desc, const deltalog_state *state, const int32_t *slot_idx,
                   int32_t n, int32_t only_if_full, void *stream) {
    if (int rc = validate_desc(desc)) return rc;
    if (int rc = validate_state(state)) return rc;
    if (n < 0 || (!slot_idx && n > desc->num_slots)) return DELTALOG_ERR_INVALID_ARG;
    if (n == 0) return DELTALOG_OK;
    const StateArgs st = make_state_args(desc, state);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    return dispatch_merge(desc, st, slot_idx, n, only_if_full, s);
}

int deltalog_reset_slots(const deltalog_desc *desc, const deltalog_state *state, const int32_t *slot_idx,
                         int32_t n, const float *S_init, void *stream) {
    if (int rc = validate_desc(desc)) return rc;
    if (int rc = validate_state(state)) return rc;
    if (n < 0 || (!slot_idx && n > desc->num_slots) || (S_init && !aligned16(S_init))) return DELTALOG_ERR_INVALID_ARG;
    if (n == 0) return DELTALOG_OK;
    const StateArgs st = make_state_args(desc, state);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    return dispatch_reset_slots(desc, st, slot_idx, n, S_init, s);
}

int deltalog_eager_step(const deltalog_desc *desc, void *S, const void *q, const void *k,
                        const void *v, const float *g, const float *beta, const float *u_bonus,
                        const int32_t *slot_idx, int32_t B, void *out, int32_t *status, void *stream) {
    if (int rc = validate_desc(desc)) return rc;
    if (!S || !aligned16(S)) return DELTALOG_ERR_INVALID_ARG;
    if (int rc = validate_token(desc, q, k, v, g, beta, u_bonus, B, out)) return rc;
    if (B == 0) return DELTALOG_OK;
    const TokenArgs tk = make_token_args(desc, q, k, v, g, beta, u_bonus, slot_idx, out, B);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    return dispatch_eager(desc, S, status, tk, s);
}

int deltalog_decode_step_host(const deltalog_desc *desc, const deltalog_state *state,
                              const deltalog_staging *staging, const void *host_q,
                              const void *host_k, const void *host_v, const float *host_g,
                              const float *host_beta, const float *u_bonus,
                              const int32_t *slot_idx, int32_t B, void *host_out, void *stream) {
    // every check of the decode step runs before the first copy is enqueued: a rejected call leaves the
    // stream and the staging buffers as they were
    if (int rc = validate_desc(desc)) return rc;
    if (int rc = validate_state(state)) return rc;
    if (!staging || !host_q || !host_k || !host_v || !host_out) return DELTALOG_ERR_INVALID_ARG;
    if (op_has_gate(desc->op) && (!host_g || !staging->g)) return DELTALOG_ERR_INVALID_ARG;
    if (op_delta_rule(desc->op) && (!host_beta || !staging->beta)) return DELTALOG_ERR_INVALID_ARG;
    if (int rc = validate_token(desc, staging->q, staging->k, staging->v, staging->g, staging->beta, u_bonus, B, staging->out))
        return rc;
    if (B == 0) return DELTALOG_OK;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t units = (size_t)B * desc->H;
    const size_t esz = desc->io_dtype == DELTALOG_F32 ? 4 : 2;
    const size_t vec = units * desc->d_v * esz;
    const size_t qk_vec = (size_t)B * qk_heads(desc) * desc->d_k * esz;
    const size_t gbytes = units * (op_vec_decay(desc->op) ? desc->d_k : 1) * sizeof(float);
    bool ok = true;
    if (const size_t block = packed_block_bytes(desc, staging, host_q, host_k, host_v, host_g, host_beta, qk_vec, vec,
                                                gbytes, units)) {
        ok = cudaMemcpyAsync(staging->q, host_q, block, cudaMemcpyHostToDevice, s) == cudaSuccess;  // one copy
    } else {
        ok = cudaMemcpyAsync(staging->q, host_q, qk_vec, cudaMemcpyHostToDevice, s) == cudaSuccess;
        ok = ok && cudaMemcpyAsync(staging->k, host_k, qk_vec, cudaMemcpyHostToDevice, s) == cudaSuccess;
        ok = ok && cudaMemcpyAsync(staging->v, host_v, vec, cudaMemcpyHostToDevice, s) == cudaSuccess;
        if (op_has_gate(desc->op))
            ok = ok && cudaMemcpyAsync(staging->g, host_g, gbytes, cudaMemcpyHostToDevice, s) == cudaSuccess;
        if (op_delta_rule(desc->op))
            ok = ok && cudaMemcpyAsync(staging->beta, host_beta, units * sizeof(float), cudaMemcpyHostToDevice, s) ==
                           cudaSuccess;
    }
    if (!ok) return DELTALOG_ERR_CUDA;
    if (int rc = deltalog_decode_step(desc, state, staging->q, staging->k, staging->v, staging->g,
                                      staging->beta, u_bonus, slot_idx, B, staging->out, stream))
        return rc;
    if (cudaMemcpyAsync(host_out, staging->out, units * desc->d_v * esz, cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return DELTALOG_ERR_CUDA;
    return DELTALOG_OK;
}

int deltalog_decode_step_host_overlapped(const deltalog_desc *desc, const deltalog_state *state,
                                         const deltalog_staging *staging, const deltalog_host_lane *lane,
                                         const void *host_q, const void *host_k, const void *host_v,
                                         const float *host_g, const float *host_beta, const float *u_bonus,
                                         const int32_t *slot_idx, int32_t B, void *host_out) {
    if (int rc = validate_desc(desc)) return rc;
    if (int rc = validate_state(state)) return rc;
    if (!staging || !lane || !host_q || !host_k || !host_v || !host_out) return DELTALOG_ERR_INVALID_ARG;
    if (!lane->in_done || !lane->compute_done || !lane->out_done) return DELTALOG_ERR_INVALID_ARG;
    if (op_has_gate(desc->op) && (!host_g || !staging->g)) return DELTALOG_ERR_INVALID_ARG;
    if (op_delta_rule(desc->op) && (!host_beta || !staging->beta)) return DELTALOG_ERR_INVALID_ARG;
    if (int rc = validate_token(desc, staging->q, staging->k, staging->v, staging->g, staging->beta, u_bonus, B, staging->out))
        return rc;
    if (B == 0) return DELTALOG_OK;
    cudaStream_t s_in = static_cast<cudaStream_t>(lane->copy_in_stream);
    cudaStream_t s_cmp = static_cast<cudaStream_t>(lane->compute_stream);
    cudaStream_t s_out = static_cast<cudaStream_t>(lane->copy_out_stream);
    cudaEvent_t e_in = static_cast<cudaEvent_t>(lane->in_done);
    cudaEvent_t e_cmp = static_cast<cudaEvent_t>(lane->compute_done);
    cudaEvent_t e_out = static_cast<cudaEvent_t>(lane->out_done);
    const size_t units = (size_t)B * desc->H;
    const size_t esz = desc->io_dtype == DELTALOG_F32 ? 4 : 2;
    const size_t vec = units * desc->d_v * esz;
    const size_t qk_vec = (size_t)B * qk_heads(desc) * desc->d_k * esz;
    const size_t gbytes = units * (op_vec_decay(desc->op) ? desc->d_k : 1) * sizeof(float);
    // copy-in stream: the staging inputs are free once the kernel that last read them is done
    bool ok = cudaStreamWaitEvent(s_in, e_cmp, 0) == cudaSuccess;
    if (const size_t block = packed_block_bytes(desc, staging, host_q, host_k, host_v, host_g, host_beta, qk_vec, vec,
                                                gbytes, units)) {
        ok = ok && cudaMemcpyAsync(staging->q, host_q, block, cudaMemcpyHostToDevice, s_in) == cudaSuccess;  // one copy
    } else {
        ok = ok && cudaMemcpyAsync(staging->q, host_q, qk_vec, cudaMemcpyHostToDevice, s_in) == cudaSuccess;
        ok = ok && cudaMemcpyAsync(staging->k, host_k, qk_vec, cudaMemcpyHostToDevice, s_in) == cudaSuccess;
        ok = ok && cudaMemcpyAsync(staging->v, host_v, vec, cudaMemcpyHostToDevice, s_in) == cudaSuccess;
        if (op_has_gate(desc->op))
            ok = ok && cudaMemcpyAsync(staging->g, host_g, gbytes, cudaMemcpyHostToDevice, s_in) == cudaSuccess;
        if (op_delta_rule(desc->op))
            ok = ok && cudaMemcpyAsync(staging->beta, host_beta, units * sizeof(float), cudaMemcpyHostToDevice, s_in) ==
                           cudaSuccess;
    }
    ok = ok && cudaEventRecord(e_in, s_in) == cudaSuccess;
    // compute stream: inputs landed, and the previous output of this staging set has been read back
    ok = ok && cudaStreamWaitEvent(s_cmp, e_in, 0) == cudaSuccess;
    ok = ok && cudaStreamWaitEvent(s_cmp, e_out, 0) == cudaSuccess;
    if (!ok) return DELTALOG_ERR_CUDA;
    if (int rc = deltalog_decode_step(desc, state, staging->q, staging->k, staging->v, staging->g,
                                      staging->beta, u_bonus, slot_idx, B, staging->out, lane->compute_stream))
        return rc;
    ok = cudaEventRecord(e_cmp, s_cmp) == cudaSuccess;
    // copy-out stream
    ok = ok && cudaStreamWaitEvent(s_out, e_cmp, 0) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(host_out, staging->out, units * desc->d_v * esz, cudaMemcpyDeviceToHost, s_out) ==
                   cudaSuccess;
    ok = ok && cudaEventRecord(e_out, s_out) == cudaSuccess;
    return ok ? DELTALOG_OK : DELTALOG_ERR_CUDA;
}

const char *deltalog_status_string(int code) {
    switch (code) {
        case DELTALOG_OK: return "ok";
        case DELTALOG_ERR_INVALID_ARG: return "invalid argument (null / misaligned pointer, bad enum or negative count)";
        case DELTALOG_ERR_UNSUPPORTED_SHAPE: return "unsupported shape or dtype combination";
        case DELTALOG_ERR_CAP_RANGE: return "log capacity outside 1..64";
        case DELTALOG_ERR_CUDA: return "CUDA runtime error";
        case DELTALOG_ERR_STATIC_LIMIT: return "request larger than the built-in staging area (DELTALOG_STATIC_STAGING_BYTES)";
        default: return "unknown status code";
    }
}

int deltalog_version(void) { return 200; }

#ifndef DELTALOG_BUILD_ID
#define DELTALOG_BUILD_ID "unknown"
#endif
const char *deltalog_build_id(void) { return DELTALOG_BUILD_ID; }

uint64_t deltalog_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
