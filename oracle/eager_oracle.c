/*
 * TEST INFRASTRUCTURE -- the parity oracle. Not part of the product path.
 *
 * Plain fp64 eager recurrence for the recurrent linear-attention operators whose
 * decode update this repository accelerates (GDN, KDA, RWKV6 and the additive
 * family of Table 1: plain linear attention, RetNet, GLA).
 * "Eager" means the dense d_k x d_v state is rewritten at every token, which is
 * the definition the deferred (base + log) schedule must reproduce exactly in
 * exact arithmetic (Section 3, Eq. 6 and the closure argument below it).
 *
 * Every function is the definition written out: no blocking, no fusion, no
 * reordering.  The state S is row-major [d_k][d_v]; the decay acts on rows
 * (the key dimension), D(l) = diag(exp(l)) (Eq. 2).
 *
 * Unified recurrence (Eq. 3):     S_t = D(lambda_t) S_{t-1} + a_t b_t^T
 * Operator table (Table 1):
 *   GDN   scalar lambda, a = k, b = beta (v - (D(lambda) S_{t-1})^T k), o = scale * S_t^T q
 *   KDA   per-key lambda, same a, b, o
 *   RWKV6 per-key lambda (log w), a = k, b = v,
 *         o = S_{t-1}^T r + (r . (bonus (.) k)) v       (readout from the pre-update state)
 *   Linear attention  no decay,         a = k (the caller applies the feature map), b = v
 *   RetNet            scalar lambda,    a = k, b = v
 *   GLA               per-key lambda,   a = k, b = v;   all three: o = scale * S_t^T q  (Eq. 3)
 *
 * Reading taken where the paper's Table 1 is ambiguous: the delta-rule
 * correction k^T S_{t-1} is evaluated on the *decayed* previous state, as the
 * text of the merge stage says ("after applying the current log-decay and
 * constructing the current update factors") and as Algorithm 1 orders its lines
 * 2 and 3.  This gives S_t = (I - beta k k^T) D(lambda) S_{t-1} + beta k v^T.
 *
 * Parity pins for every function here live in tests/test_oracle_pins.py
 * (closed forms, invariants, special cases); nothing is "parity unpinned".
 *
 * Build: gcc -O2 -fopenmp -shared -fPIC eager_oracle.c -o liboracle.so -lm
 */
#include <math.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* The value a 16-bit (bfloat16) state element holds after a store of x: fp64 -> fp32 -> bfloat16, both
 * round-to-nearest-even (the 16-bit-state variant of the roofline discussion in Section 2.2; the
 * arithmetic of a token stays fp64, only what is kept between tokens is rounded).  Finite x only. */
static double round_to_bf16(double x)
{
    float f = (float)x;
    unsigned int u;
    memcpy(&u, &f, sizeof u);
    u = (u + 0x7fffu + ((u >> 16) & 1u)) & 0xffff0000u;
    memcpy(&f, &u, sizeof u);
    return (double)f;
}

enum { ORACLE_GDN = 0, ORACLE_KDA = 1, ORACLE_RWKV6 = 2, ORACLE_LINATTN = 3, ORACLE_RETNET = 4, ORACLE_GLA = 5 };

/* One token of the gated delta rule (GDN: d_lambda == 1, KDA: d_lambda == d_k). */
static void delta_rule_token(int d_k, int d_v, int d_lambda, double scale, double *S,
                             const double *q, const double *k, const double *v,
                             const double *lambda, double beta, double *o, double *b)
{
    int j, c;
    /* state transform S' = D(lambda_t) S_{t-1}   (Eq. 3) */
    for (j = 0; j < d_k; ++j) {
        double a = exp(lambda[d_lambda == 1 ? 0 : j]);
        for (c = 0; c < d_v; ++c) S[(size_t)j * d_v + c] *= a;
    }
    /* value-side factor b_t = beta_t (v_t - S'^T k_t)   (Table 1, rows GDN / KDA) */
    for (c = 0; c < d_v; ++c) {
        double corr = 0.0;
        for (j = 0; j < d_k; ++j) corr += S[(size_t)j * d_v + c] * k[j];
        b[c] = beta * (v[c] - corr);
    }
    /* rank-one update S_t = S' + k_t b_t^T   (Eq. 3 with a_t = k_t) */
    for (j = 0; j < d_k; ++j)
        for (c = 0; c < d_v; ++c) S[(size_t)j * d_v + c] += k[j] * b[c];
    /* readout from the updated state o_t = scale * S_t^T q_t   (Eq. 3) */
    for (c = 0; c < d_v; ++c) {
        double acc = 0.0;
        for (j = 0; j < d_k; ++j) acc += S[(size_t)j * d_v + c] * q[j];
        o[c] = scale * acc;
    }
}

/* One token of the additive family (Table 1: linear attention d_lambda == 0, RetNet d_lambda == 1,
 * GLA d_lambda == d_k): S_t = D(lambda_t) S_{t-1} + k_t v_t^T, o_t = scale * S_t^T q_t   (Eq. 3). */
static void additive_token(int d_k, int d_v, int d_lambda, double scale, double *S, const double *q,
                           const double *k, const double *v, const double *lambda, double *o, double *b)
{
    int j, c;
    for (j = 0; j < d_k; ++j) {
        double a = d_lambda == 0 ? 1.0 : exp(lambda[d_lambda == 1 ? 0 : j]);
        for (c = 0; c < d_v; ++c) S[(size_t)j * d_v + c] = a * S[(size_t)j * d_v + c] + k[j] * v[c];
    }
    for (c = 0; c < d_v; ++c) {
        double acc = 0.0;
        for (j = 0; j < d_k; ++j) acc += S[(size_t)j * d_v + c] * q[j];
        o[c] = scale * acc;
        b[c] = v[c];
    }
}

/* One token of RWKV6: readout first (pre-update state plus the bonus term), then update. */
static void rwkv6_token(int d_k, int d_v, double *S, const double *r, const double *k,
                        const double *v, const double *log_w, const double *bonus, double *o,
                        double *b)
{
    int j, c;
    double rk = 0.0;
    for (j = 0; j < d_k; ++j) rk += r[j] * bonus[j] * k[j];
    /* o_t = S_{t-1}^T r_t + (r_t . (bonus (.) k_t)) v_t */
    for (c = 0; c < d_v; ++c) {
        double acc = 0.0;
        for (j = 0; j < d_k; ++j) acc += S[(size_t)j * d_v + c] * r[j];
        o[c] = acc + rk * v[c];
    }
    /* S_t = diag(w_t) S_{t-1} + k_t v_t^T   (Table 1, row RWKV6; w_t = exp(log_w)) */
    for (j = 0; j < d_k; ++j) {
        double w = exp(log_w[j]);
        for (c = 0; c < d_v; ++c)
            S[(size_t)j * d_v + c] = w * S[(size_t)j * d_v + c] + k[j] * v[c];
    }
    for (c = 0; c < d_v; ++c) b[c] = v[c];
}

/*
 * Roll T tokens through N independent (sequence, head) units.
 *
 *   S        [N][d_k][d_v]   in: S_0, out: S_T (updated in place)
 *   q, k     [T][N][d_k]     (q is r for RWKV6)
 *   v        [T][N][d_v]
 *   lambda   [T][N][d_lambda] log-decay, d_lambda = 1 (GDN, RetNet) or d_k (KDA, RWKV6, GLA);
 *                            ignored (may be NULL) for plain linear attention
 *   beta     [T][N]          GDN / KDA only (may be NULL for RWKV6)
 *   bonus    [N][d_k]        RWKV6 only (may be NULL otherwise)
 *   out      [T][N][d_v]
 *   b_rec    [T][N][d_v]     the value-side factor b_t of every token, or NULL
 *   snap_at  [n_snap]        ascending 1-based token counts after which S is recorded
 *   S_snap   [n_snap][N][d_k][d_v]
 *   state_bf16               nonzero: the state is kept in bfloat16 between tokens (rounded after every
 *                            token's update; the token's output is formed before the rounding)
 *
 * Units run in parallel (OpenMP); each keeps its state hot across its T tokens.
 * Returns 0, or -1 for an unknown operator.
 */
int oracle_eager_rollout(int op, int T, int N, int d_k, int d_v, double scale, double *S,
                         const double *q, const double *k, const double *v, const double *lambda,
                         const double *beta, const double *bonus, double *out, double *b_rec,
                         int n_snap, const int *snap_at, double *S_snap, int state_bf16)
{
    int d_lambda = (op == ORACLE_GDN || op == ORACLE_RETNET) ? 1 : (op == ORACLE_LINATTN ? 0 : d_k);
    int n;
    if (op < ORACLE_GDN || op > ORACLE_GLA) return -1;
#pragma omp parallel for schedule(dynamic, 1)
    for (n = 0; n < N; ++n) {
        double *Sn = S + (size_t)n * d_k * d_v;
        double *b_tmp = (double *)malloc(sizeof(double) * (size_t)d_v);
        int t, next_snap = 0;
        for (t = 0; t < T; ++t) {
            size_t tn = (size_t)t * N + n;
            double *o = out + tn * d_v;
            double *b = b_rec ? b_rec + tn * d_v : b_tmp;
            if (op == ORACLE_RWKV6)
                rwkv6_token(d_k, d_v, Sn, q + tn * d_k, k + tn * d_k, v + tn * d_v,
                            lambda + tn * d_lambda, bonus + (size_t)n * d_k, o, b);
            else if (op >= ORACLE_LINATTN)
                additive_token(d_k, d_v, d_lambda, scale, Sn, q + tn * d_k, k + tn * d_k, v + tn * d_v,
                               d_lambda ? lambda + tn * d_lambda : NULL, o, b);
            else
                delta_rule_token(d_k, d_v, d_lambda, scale, Sn, q + tn * d_k, k + tn * d_k,
                                 v + tn * d_v, lambda + tn * d_lambda, beta[tn], o, b);
            if (state_bf16) {
                size_t x;
                for (x = 0; x < (size_t)d_k * d_v; ++x) Sn[x] = round_to_bf16(Sn[x]);
            }
            while (next_snap < n_snap && snap_at[next_snap] == t + 1) {
                memcpy(S_snap + ((size_t)next_snap * N + n) * d_k * d_v, Sn,
                       sizeof(double) * (size_t)d_k * d_v);
                ++next_snap;
            }
        }
        free(b_tmp);
    }
    return 0;
}

/* Number of host threads oracle_eager_rollout will use. */
int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
