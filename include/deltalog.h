/*
 * deltalog.h -- C ABI of the DeltaLog recurrent-state decode library (sm_100a).
 *
 * The library keeps the recurrent state of a linear-attention layer as a dense base (fp32; bf16 as an
 * option, see deltalog_desc.base_dtype) plus a
 * bounded log of compact per-token factors (Section 3.1 of the paper):
 *
 *     S_t = D(lbar) S_base + sum_{i < len} D(lbar - Lambda[i]) K[i] U[i]^T          (Eq. 6)
 *
 * with D(l) = diag(exp(l)) acting on the key dimension (rows), lbar the log-decay accumulated
 * since the last materialisation and Lambda[i] its snapshot when entry i was appended.  Because
 * Lambda[len-1] is lbar by construction (Eq. 4 stores lbar after it absorbed the token's decay),
 * lbar is not stored separately: lbar = Lambda[len-1], or 0 for an empty log.
 *
 * Operators (Table 1; the gate is passed in log space, lambda_t = log alpha_t or log w_t):
 *   DELTALOG_GDN    scalar decay per head, delta rule:   b_t = beta_t (v_t - (D(lambda_t) S_{t-1})^T k_t)
 *   DELTALOG_KDA    per-key decay,          delta rule:   same b_t
 *   DELTALOG_RWKV6  per-key decay, b_t = v_t, output read from S_{t-1} plus the bonus term
 *   DELTALOG_LINATTN  no decay (the gate pointer is ignored and may be NULL), b_t = v_t; the caller
 *                     passes the feature-mapped key phi(k_t) as k
 *   DELTALOG_RETNET   scalar decay per head (lambda = log gamma), b_t = v_t
 *   DELTALOG_GLA      per-key decay, b_t = v_t
 * All use a_t = k_t and S_t = D(lambda_t) S_{t-1} + a_t b_t^T (Eq. 3); all but RWKV6 return
 * scale * S_t^T q_t.  beta is read by GDN / KDA only, u_bonus by RWKV6 only.
 *
 * General rules for every entry point
 *   - All tensor pointers are DEVICE pointers owned by the caller; descriptor structs are HOST
 *     memory, read during the call only.  The library allocates nothing and keeps no state about
 *     the caller's tensors (it only remembers, per device, facts it queried and kernel attributes it
 *     set).
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*, NULL = default stream)
 *     and never synchronise.
 *   - Tensors are dense, row-major in the index order written beside them, 16-byte aligned.
 *   - Return value: DELTALOG_OK (0) when the work was launched; any other code means the
 *     arguments were rejected on the host and nothing was launched.
 *   - Conditions only visible on the device (a row whose log is already full, a slot index out of
 *     range) make the kernel skip that row, OR a bit into *state->status (if non-NULL) and carry
 *     on; kernels never trap.  Rows with slot index < 0 are padding and are skipped silently.
 *   - The same slot must not appear twice in one call.
 *   - Supported shapes: d_k and d_v each 64 or 128 (they may differ: the tile is d_k rows x d_v columns;
 *     q, k, the gate of the per-key operators and K_log are d_k wide, v, out and U_log d_v wide);
 *     1 <= cap <= 64; klog_dtype == io_dtype;
 *     ulog_dtype == io_dtype for the operators with b_t = v_t; F32 for GDN / KDA (the paper keeps b_t in
 *     fp32 against cancellation in the correction path), or, as a reduced-precision variant that does
 *     NOT meet the 1e-4 state tolerance, == io_dtype == BF16.
 */
#ifndef DELTALOG_H
#define DELTALOG_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DELTALOG_GDN = 0, DELTALOG_KDA = 1, DELTALOG_RWKV6 = 2, DELTALOG_LINATTN = 3, DELTALOG_RETNET = 4, DELTALOG_GLA = 5
} deltalog_op;
typedef enum { DELTALOG_F32 = 0, DELTALOG_BF16 = 1 } deltalog_dtype;

/* host-side return codes */
enum {
    DELTALOG_OK = 0,
    DELTALOG_ERR_INVALID_ARG = 1,       /* NULL where a pointer is required, B < 0, bad enum, misaligned pointer */
    DELTALOG_ERR_UNSUPPORTED_SHAPE = 2, /* d_k / d_v / dtype combination outside the supported set */
    DELTALOG_ERR_CAP_RANGE = 3,         /* cap outside 1..64 */
    DELTALOG_ERR_CUDA = 4,              /* the CUDA runtime refused the launch or a copy */
    DELTALOG_ERR_STATIC_LIMIT = 5       /* the request does not fit the built-in staging area (see below) */
};

/* bits OR-ed into *status by kernels */
enum {
    DELTALOG_STATUS_LOG_FULL = 1, /* decode on a (slot, head) whose log already holds cap entries: row skipped */
    DELTALOG_STATUS_BAD_SLOT = 2, /* slot index >= num_slots: row skipped */
    DELTALOG_STATUS_TIMEOUT = 4   /* a bounded wait inside a kernel gave up: results of that launch are invalid */
};

/* Problem description (host memory). */
typedef struct {
    int32_t op;         /* deltalog_op */
    int32_t num_slots;  /* size of the state pool */
    int32_t H;          /* heads */
    int32_t d_k, d_v;   /* head dimensions */
    int32_t cap;        /* log capacity: appends possible between two merges */
    int32_t io_dtype;   /* deltalog_dtype of q, k, v, out */
    int32_t klog_dtype; /* deltalog_dtype of K_log */
    int32_t ulog_dtype; /* deltalog_dtype of U_log */
    float scale;        /* multiplies the output of GDN / KDA (ignored for RWKV6) */
    int32_t H_qk;       /* query/key heads: 0 or H = one per state head; otherwise a divisor of H, and state
                           head h uses the q and k of head h / (H / H_qk) (grouped heads: several value
                           heads share one query/key head); q and k are then [B, H_qk, d_k] */
    int32_t hints;      /* DELTALOG_HINT_* bits, 0 = none */
    int32_t base_dtype; /* deltalog_dtype of the dense state: S_base, and S of deltalog_eager_step.
                           DELTALOG_F32 (0, the default) or DELTALOG_BF16 -- the 16-bit state of the
                           roofline discussion (Section 2.2): half the dense bytes.  All arithmetic stays
                           fp32; a bf16 state is rounded (to nearest even) only when the dense state is
                           written: once per materialisation with the log schedule (Eq. 5), once per
                           token with the eager step.  Requires io_dtype == DELTALOG_BF16. */
} deltalog_desc;

/*
 * Hints (deltalog_desc.hints).  A hint is a promise by the caller; breaking it is a data race.  The paper
 * has no counterpart; the hints remove the ramp-up and tail of back-to-back decode launches (a few
 * microseconds each).
 *   DELTALOG_HINT_BASE_UNTOUCHED  The work queued on the stream directly in front of this
 *       deltalog_decode_step does not WRITE S_base of the slots this call reads.  (True when it was
 *       another decode step on this state, or the kernel that produced this step's q, k, v, g, beta;
 *       NOT true for deltalog_merge, deltalog_decode_merge_step, deltalog_reset_slots or
 *       deltalog_eager_step on these slots.)  The decode kernel is then launched with programmatic
 *       stream serialisation: its CTAs may start while the preceding kernel is still retiring.  Ahead of
 *       that kernel's completion they read base tiles and nothing else -- unless the next hint allows the
 *       slot list too.  Everything else this call reads (q, k, v, g, beta, u_bonus, lengths, log
 *       entries) is read only after the preceding kernel has completed and its writes are visible, so
 *       the preceding kernel may well be the one that writes those tensors.
 *   DELTALOG_HINT_SLOTS_STABLE    In addition: the work directly in front does not write slot_idx
 *       either.  Base tiles are addressed through slot_idx, so with a non-NULL slot_idx the early start
 *       above streams tiles only under this second promise; without it the kernel still overlaps its
 *       launch latency with the preceding kernel but waits before its first read.  With slot_idx == NULL
 *       the bit changes nothing.
 *   DELTALOG_HINT_WALK_DOWN       No promise, an ordering request: the persistent decode kernels take the
 *       call's (row, head) units from the last to the first instead of from the first to the last.  The
 *       results are the same bit for bit (a unit's arithmetic does not depend on its place in the walk).
 *       A caller that sets the bit on every other step of a state lets each step begin with the base
 *       tiles the step before read last, which are still in L2 (configuration 1: -1.7 % per step).
 *       deltalog_merge and deltalog_decode_merge_step walk downwards by themselves, so the step after
 *       one of them should walk upwards.  deltalog_eager_step honours the bit as well (its CTAs are
 *       numbered downwards: a step then begins with the tiles the step before wrote last); the other
 *       kernels with one CTA per unit ignore it.
 */
enum { DELTALOG_HINT_BASE_UNTOUCHED = 1, DELTALOG_HINT_SLOTS_STABLE = 2, DELTALOG_HINT_WALK_DOWN = 4 };

/* Physical state (Section 3.1).  Device pointers, caller-owned. d_lambda = 1 (GDN) or d_k. */
typedef struct {
    void *S_base;      /* [num_slots, H, d_k, d_v] dense base, fp32 (or desc.base_dtype)            */
    void *K_log;       /* [num_slots, H, cap, d_k] key-side factors a_t                             */
    void *U_log;       /* [num_slots, H, cap, d_v] value-side factors b_t                           */
    float *decay_log;  /* [num_slots, H, cap, d_lambda] Lambda: cumulative log-decay snapshots, fp32 */
    int32_t *log_len;  /* [num_slots, H] live entries, 0..cap; zero it for a fresh or reused slot   */
    int32_t *status;   /* one word of DELTALOG_STATUS_* bits, or NULL                               */
} deltalog_state;

/*
 * One decode token for B rows (Algorithm 1, append branch; Eq. 4).
 * Row b updates slot slot_idx[b] (slot b if slot_idx is NULL), all H heads.
 * Reads S_base once and the live log entries; computes `out`; appends (k_t, b_t, lbar + lambda_t)
 * as entry log_len and increments log_len.  Never writes S_base.
 *
 *   q, k, v  [B, H, d]  io_dtype (q is the receptance r for RWKV6)
 *   q, k     [B, H_qk, d_k] io_dtype (H_qk = H unless the descriptor groups heads); v [B, H, d_v]
 *   g        log-decay lambda_t <= 0, fp32: [B, H] for GDN / RetNet, [B, H, d_k] for KDA / RWKV6 / GLA;
 *            ignored (may be NULL) for plain linear attention
 *   beta     [B, H] fp32 for GDN / KDA; ignored (may be NULL) otherwise
 *   u_bonus  [H, d_k] fp32 for RWKV6; ignored (may be NULL) otherwise
 *   out      [B, H, d_v] io_dtype;  GDN / KDA: scale * S_t^T q_t;
 *            RWKV6: S_{t-1}^T r_t + (r_t . (u_bonus (.) k_t)) v_t
 */
int deltalog_decode_step(const deltalog_desc *desc, const deltalog_state *state, const void *q,
                         const void *k, const void *v, const float *g, const float *beta,
                         const float *u_bonus, const int32_t *slot_idx, int32_t B, void *out,
                         void *stream);

/*
 * T consecutive tokens for each of the B rows in one call (several tokens of a request at once, e.g.
 * the verification step of speculative decoding).  Results are those of T successive
 * deltalog_decode_step calls; the base tile is read once for all T tokens.  Token tensors carry a
 * token axis after the batch axis: q, k [B, T, H_qk, d_k]; v, out [B, T, H, d_v]; g [B, T, H] or
 * [B, T, H, d_k]; beta [B, T, H].  1 <= T <= cap (DELTALOG_ERR_CAP_RANGE otherwise).  A (row, head)
 * whose log has no room for all T entries (log_len + T > cap) is skipped as a whole -- nothing is
 * appended, `out` is not written -- and DELTALOG_STATUS_LOG_FULL is raised.  The paper's decode path
 * is single-token; this entry point extends its append branch (Algorithm 1) to a block of tokens.
 */
int deltalog_decode_steps(const deltalog_desc *desc, const deltalog_state *state, const void *q, const void *k,
                          const void *v, const float *g, const float *beta, const float *u_bonus,
                          const int32_t *slot_idx, int32_t B, int32_t T, void *out, void *stream);

/*
 * The merge step of the cycle as the paper runs it (Algorithm 1, else-branch; Eq. 5 with the
 * current-token term): every row of the batch consumes its token AND has its state materialised,
 *     lbar <- lbar + lambda_t ;  (a_t, b_t) and `out` exactly as in deltalog_decode_step ;
 *     S_base <- D(lbar) S_base + sum_i D(lbar - Lambda[i]) K[i] U[i]^T + a_t b_t^T ;  log_len <- 0
 * whatever the live length of its log (0..cap; with an empty log this is the eager step on S_base).
 * The token is NOT appended.  Arguments, layouts and status bits as for deltalog_decode_step;
 * DELTALOG_STATUS_LOG_FULL is never raised.  The caller keeps phase-split batches (Section 4):
 * rows whose log is full go through this call, the others through deltalog_decode_step.  One read
 * and one write of each listed row's base tile.
 */
int deltalog_decode_merge_step(const deltalog_desc *desc, const deltalog_state *state, const void *q,
                               const void *k, const void *v, const float *g, const float *beta,
                               const float *u_bonus, const int32_t *slot_idx, int32_t B, void *out,
                               void *stream);

/*
 * Materialise the log into the base (Eq. 5 without the current-token term):
 *     S_base <- D(lbar) S_base + sum_i D(lbar - Lambda[i]) K[i] U[i]^T ;  log_len <- 0
 * for the n slots listed in slot_idx (slots 0..n-1 if NULL), all heads.  A (slot, head) with an
 * empty log is left untouched (no dense write).  With only_if_full != 0, (slot, head) pairs whose
 * log holds fewer than cap entries are skipped as well, so one call over the whole batch serves
 * sequences whose merge boundaries are staggered.
 */
int deltalog_merge(const deltalog_desc *desc, const deltalog_state *state, const int32_t *slot_idx,
                   int32_t n, int32_t only_if_full, void *stream);

/*
 * Slot lifecycle (Section 4, state-slot lifecycle): hand the n listed slots (slots 0..n-1 if slot_idx
 * is NULL) to new requests.  The log of every head of a listed slot is emptied (log_len <- 0, which
 * also clears lbar); pending entries are discarded, not folded.  With S_init != NULL (device,
 * [n, H, d_k, d_v] fp32, e.g. the state a prefill produced) the base of listed slot i becomes
 * S_init[i] (rounded to desc.base_dtype where that is 16-bit); with S_init == NULL the base is left as it is.  Other slots are untouched.  Slot
 * indices < 0 are skipped, indices >= num_slots set DELTALOG_STATUS_BAD_SLOT and are skipped.
 */
int deltalog_reset_slots(const deltalog_desc *desc, const deltalog_state *state, const int32_t *slot_idx,
                         int32_t n, const float *S_init, void *stream);

/*
 * The eager dense comparator (Section 2.3): the same token update applied directly to a dense
 * state S [num_slots, H, d_k, d_v] (fp32, or desc.base_dtype), read and rewritten in full on every call.
 * Token arguments and `out` as for deltalog_decode_step; `status` (may be NULL) receives
 * DELTALOG_STATUS_BAD_SLOT bits.
 */
int deltalog_eager_step(const deltalog_desc *desc, void *S, const void *q, const void *k,
                        const void *v, const float *g, const float *beta, const float *u_bonus,
                        const int32_t *slot_idx, int32_t B, void *out, int32_t *status, void *stream);

/*
 * deltalog_decode_step for callers whose token tensors live in HOST memory (pinned for the copies
 * to be asynchronous): copies q, k, v, g, beta (and nothing else) to the caller-provided device
 * staging buffers on `stream`, runs the decode step there and copies `out` back to host_out.
 * The state, u_bonus and slot_idx stay device-resident.  Staging buffers have the shapes of the
 * tensors they stage.  Returns after enqueuing; synchronise the stream before reading host_out.
 * Packed buffers (staging->packed != 0): q, k, v, g (operators with a gate) and beta (delta rule)
 * follow one another in this order, each starting on the next 256-byte boundary after the previous
 * one ends, inside one allocation -- in host memory AND in the staging buffers alike.  The copies then
 * collapse into one over the whole block (small host-to-device copies run far below the link rate).
 * If the pointers do not have that layout the flag is ignored and every tensor is copied on its own.
 */
typedef struct {
    void *q, *k, *v; /* device, [B, H, d] io_dtype */
    float *g;        /* device, shape of g */
    float *beta;     /* device, [B, H]; unused for RWKV6 */
    void *out;       /* device, [B, H, d_v] io_dtype */
    int32_t packed;  /* != 0: the caller promises that q, k, v, g, beta are carved out of ONE allocation in
                        the packed layout described below, here and in host memory alike */
} deltalog_staging;

int deltalog_decode_step_host(const deltalog_desc *desc, const deltalog_state *state,
                              const deltalog_staging *staging, const void *host_q,
                              const void *host_k, const void *host_v, const float *host_g,
                              const float *host_beta, const float *u_bonus,
                              const int32_t *slot_idx, int32_t B, void *host_out, void *stream);

/*
 * deltalog_decode_step_host with the three phases of a step on three streams, so that the copies
 * of consecutive steps overlap the kernels: while step t runs on compute_stream, the token tensors
 * of step t+1 are already being copied in and the output of step t-1 is being copied out.  The
 * caller owns the streams and the events and alternates between (at least) two sets of
 * {staging, in_done, compute_done, out_done}; the streams are shared by all sets.  Per call:
 *     copy_in_stream :  wait compute_done (the kernel that last read this staging set);  H2D copies
 *                       of q, k, v, g, beta;  record in_done
 *     compute_stream :  wait in_done and out_done (previous read-back of this set);  decode kernel;
 *                       record compute_done
 *     copy_out_stream:  wait compute_done;  D2H copy of out into host_out;  record out_done
 * Kernels of consecutive steps (and the caller's deltalog_merge calls, which belong on
 * compute_stream) stay ordered because they share compute_stream.  Synchronise out_done before
 * reading host_out.  Events must have been created by the caller; an event that was never recorded
 * is treated as complete.  Other arguments and return codes as deltalog_decode_step_host.
 */
typedef struct {
    void *copy_in_stream, *compute_stream, *copy_out_stream; /* cudaStream_t */
    void *in_done, *compute_done, *out_done;                 /* cudaEvent_t, one triple per staging set */
} deltalog_host_lane;

int deltalog_decode_step_host_overlapped(const deltalog_desc *desc, const deltalog_state *state,
                                         const deltalog_staging *staging, const deltalog_host_lane *lane,
                                         const void *host_q, const void *host_k, const void *host_v,
                                         const float *host_g, const float *host_beta, const float *u_bonus,
                                         const int32_t *slot_idx, int32_t B, void *host_out);

/*
 * (No counterpart in the paper: a convenience for callers that must not allocate.)
 *
 * deltalog_decode_step_host without the staging argument.  Some callers cannot provide device
 * staging buffers because they are not allowed to call cudaMalloc -- code that runs inside a
 * latency-critical serving loop where an allocation may synchronise the device, plug-ins that are
 * handed a stream but no allocator, or a process whose memory pool is owned by another component.
 * For them the staging area is a fixed array inside the library (DELTALOG_STATIC_STAGING_BYTES of
 * device memory on every GPU that loads the library, held until the process exits); this call
 * allocates nothing, frees nothing and calls no allocating library routine.
 *
 *   - Limit: the staged tensors (q, k, v, g, beta, out, each rounded up to 256 bytes) must fit in
 *     DELTALOG_STATIC_STAGING_BYTES; e.g. bf16, H = 32, d = 128 allows B <= 254 for GDN.  Larger
 *     requests return DELTALOG_ERR_STATIC_LIMIT and nothing is enqueued.
 *   - The first call on each device looks up the array's device address (with that device
 *     current).  Make that first call before any stream capture begins.
 *   - All calls on a device share the one array.  Two calls whose GPU work may overlap (different
 *     streams, or a call issued before the previous host_out was consumed on another stream)
 *     race on it; serialise them.  The array keeps the previous call's contents; the output part
 *     is cleared at the start of every call, so rows the kernel skips (slot < 0, bad slot, full
 *     log) read back as zeros in host_out.
 *   - Arguments, results and return codes otherwise exactly as deltalog_decode_step_host.
 */
#define DELTALOG_STATIC_STAGING_BYTES (8u << 20)
int deltalog_decode_step_host_static(const deltalog_desc *desc, const deltalog_state *state,
                                     const void *host_q, const void *host_k, const void *host_v,
                                     const float *host_g, const float *host_beta, const float *u_bonus,
                                     const int32_t *slot_idx, int32_t B, void *host_out, void *stream);

/* Human-readable text for a host return code (static storage). */
const char *deltalog_status_string(int code);

/* Library version, major * 10000 + minor * 100 + patch. */
int deltalog_version(void);

/* Identifier of the sources and compiler switches this library was built from (static storage; "unknown"
 * when the build did not supply one).  Profiler figures stored beside the code carry the identifier of the
 * build they were captured on. */
const char *deltalog_build_id(void);

/* Number of kernels the library has launched in this process (host counter, all entry points). */
uint64_t deltalog_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* DELTALOG_H */
