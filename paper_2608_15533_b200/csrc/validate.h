// Host-side argument checks shared by the entry points (every translation unit of the library that
// takes caller arguments runs them before it enqueues anything).
#pragma once

#include <cstdint>

#include "deltalog.h"

namespace deltalog {

constexpr int kMaxCapHost = 64;

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Operator facts needed on the host side (Table 1).
inline bool op_delta_rule(int op) { return op == DELTALOG_GDN || op == DELTALOG_KDA; }
inline bool op_has_gate(int op) { return op != DELTALOG_LINATTN; }
inline bool op_vec_decay(int op) { return op == DELTALOG_KDA || op == DELTALOG_RWKV6 || op == DELTALOG_GLA; }

inline int validate_desc(const deltalog_desc *d) {
    if (!d) return DELTALOG_ERR_INVALID_ARG;
    if (d->op < DELTALOG_GDN || d->op > DELTALOG_GLA) return DELTALOG_ERR_INVALID_ARG;
    if (d->num_slots <= 0 || d->H <= 0) return DELTALOG_ERR_INVALID_ARG;
    if (d->H_qk < 0 || (d->H_qk > 0 && d->H % d->H_qk != 0)) return DELTALOG_ERR_INVALID_ARG;
    if (d->io_dtype != DELTALOG_F32 && d->io_dtype != DELTALOG_BF16) return DELTALOG_ERR_INVALID_ARG;
    if (d->klog_dtype != DELTALOG_F32 && d->klog_dtype != DELTALOG_BF16) return DELTALOG_ERR_INVALID_ARG;
    if (d->ulog_dtype != DELTALOG_F32 && d->ulog_dtype != DELTALOG_BF16) return DELTALOG_ERR_INVALID_ARG;
    if ((d->d_k != 64 && d->d_k != 128) || (d->d_v != 64 && d->d_v != 128)) return DELTALOG_ERR_UNSUPPORTED_SHAPE;
    if (d->klog_dtype != d->io_dtype) return DELTALOG_ERR_UNSUPPORTED_SHAPE;
    // b = v is lossless in the I/O dtype; the delta rule keeps b in fp32 unless the caller asks for the
    // reduced-precision 16-bit U log (only with 16-bit I/O)
    const bool u_ok = op_delta_rule(d->op) ? (d->ulog_dtype == DELTALOG_F32 || d->ulog_dtype == d->io_dtype)
                                           : d->ulog_dtype == d->io_dtype;
    if (!u_ok) return DELTALOG_ERR_UNSUPPORTED_SHAPE;
    if (d->cap < 1 || d->cap > kMaxCapHost) return DELTALOG_ERR_CAP_RANGE;
    if (d->base_dtype != DELTALOG_F32 && d->base_dtype != DELTALOG_BF16) return DELTALOG_ERR_INVALID_ARG;
    // the 16-bit dense state is built for the 16-bit I/O configurations only
    if (d->base_dtype == DELTALOG_BF16 && d->io_dtype != DELTALOG_BF16) return DELTALOG_ERR_UNSUPPORTED_SHAPE;
    return DELTALOG_OK;
}

inline int validate_state(const deltalog_state *s) {
    if (!s || !s->S_base || !s->K_log || !s->U_log || !s->decay_log || !s->log_len)
        return DELTALOG_ERR_INVALID_ARG;
    if (!aligned16(s->S_base) || !aligned16(s->K_log) || !aligned16(s->U_log) || !aligned16(s->decay_log))
        return DELTALOG_ERR_INVALID_ARG;
    return DELTALOG_OK;
}

inline int validate_token(const deltalog_desc *d, const void *q, const void *k, const void *v, const float *g,
                   const float *beta, const float *u_bonus, int32_t B, const void *out) {
    if (B < 0) return DELTALOG_ERR_INVALID_ARG;
    if (!q || !k || !v || !out) return DELTALOG_ERR_INVALID_ARG;
    if (op_has_gate(d->op) && !g) return DELTALOG_ERR_INVALID_ARG;
    if (op_delta_rule(d->op) && !beta) return DELTALOG_ERR_INVALID_ARG;
    if (d->op == DELTALOG_RWKV6 && !u_bonus) return DELTALOG_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || (op_has_gate(d->op) && !aligned16(g)))
        return DELTALOG_ERR_INVALID_ARG;
    return DELTALOG_OK;
}

}  // namespace deltalog
