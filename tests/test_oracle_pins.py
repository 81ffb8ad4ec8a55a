"""Pins for the CPU oracle: closed forms, invariants and special cases fixed by the paper and by
linear algebra.  None of the expected values below is produced by the oracle's own arithmetic.

What each pin would catch:
  * explicit product of (I - beta k k^T) D(lambda) factors  -> wrong order of decay / correction /
    update, decay applied to columns instead of rows, wrong sign in the correction;
  * unrolled sum of outer products for RWKV6                -> decay applied to the new token,
    readout taken after instead of before the update, bonus on the wrong operand;
  * identity / pure-decay invariants, delta-rule recall     -> dropped terms, beta misplaced;
  * KDA with equal channels == GDN, superposition           -> per-key indexing, hidden non-linearity;
  * Eq. 1 prefix sums                                       -> transposed state (k v^T vs v k^T).
"""
import numpy as np
import pytest

import oracle
from oracle import GDN, GLA, KDA, LINATTN, RETNET, RWKV6, logical

ALL_OPS = [GDN, KDA, RWKV6, LINATTN, RETNET, GLA]

RNG = np.random.default_rng(12345)


def rand_inputs(op, T, N, dk, dv, rng=None, unit_keys=False):
    rng = rng or np.random.default_rng(T * 1000 + N * 100 + dk * 10 + dv + op)
    dl = 1 if op in (GDN, RETNET, LINATTN) else dk
    S0 = rng.normal(0, 0.3, (N, dk, dv))
    q = rng.normal(0, 1, (T, N, dk))
    k = rng.normal(0, 1, (T, N, dk))
    if unit_keys:
        k /= np.linalg.norm(k, axis=-1, keepdims=True)
    v = rng.normal(0, 1, (T, N, dv))
    lam = -np.log1p(np.exp(rng.normal(0, 1, (T, N, dl))))
    if op == LINATTN:
        lam = np.zeros((T, N, 1))   # plain linear attention has no decay
    beta = 1 / (1 + np.exp(-rng.normal(0, 1, (T, N))))
    bonus = rng.normal(0, 0.5, (N, dk))
    return S0, q, k, v, lam, beta, bonus


def roll(op, S0, q, k, v, lam, beta, bonus, **kw):
    if op == RWKV6:
        return oracle.eager_rollout(op, S0, q, k, v, lam, bonus=bonus, **kw)
    if op in (LINATTN, RETNET, GLA):
        return oracle.eager_rollout(op, S0, q, k, v, lam, **kw)
    return oracle.eager_rollout(op, S0, q, k, v, lam, beta=beta, **kw)


# ---------------------------------------------------------------------------------------------
# GDN / KDA: explicit dense transition matrices A_s = (I - beta_s k_s k_s^T) D(lambda_s)
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("op", [GDN, KDA])
@pytest.mark.parametrize("T,dk,dv", [(1, 2, 3), (5, 4, 3), (8, 8, 5), (7, 3, 8)])
def test_delta_rule_matches_explicit_product_of_factors(op, T, dk, dv):
    N = 3
    S0, q, k, v, lam, beta, _ = rand_inputs(op, T, N, dk, dv)
    scale = 0.7
    res = oracle.eager_rollout(op, S0, q, k, v, lam, beta=beta, scale=scale,
                               snapshot_at=range(1, T + 1))
    for n in range(N):
        A = []
        for s in range(T):
            dvec = np.exp(np.broadcast_to(lam[s, n], (dk,)))
            A.append((np.eye(dk) - beta[s, n] * np.outer(k[s, n], k[s, n])) @ np.diag(dvec))
        for t in range(1, T + 1):
            P = np.eye(dk)
            for s in range(t):
                P = A[s] @ P
            S_t = P @ S0[n]
            for s in range(t):
                Q = np.eye(dk)
                for r in range(s + 1, t):
                    Q = A[r] @ Q
                S_t = S_t + Q @ (beta[s, n] * np.outer(k[s, n], v[s, n]))
            np.testing.assert_allclose(res["snapshots"][t - 1, n], S_t, rtol=0, atol=1e-12)
            np.testing.assert_allclose(res["out"][t - 1, n], scale * (S_t.T @ q[t - 1, n]),
                                       rtol=0, atol=1e-12)
        np.testing.assert_allclose(res["S"][n], res["snapshots"][T - 1, n], rtol=0, atol=0)


@pytest.mark.parametrize("op", [GDN, KDA])
def test_value_side_factor_is_beta_times_residual_on_decayed_state(op):
    T, N, dk, dv = 4, 2, 5, 6
    S0, q, k, v, lam, beta, _ = rand_inputs(op, T, N, dk, dv)
    res = oracle.eager_rollout(op, S0, q, k, v, lam, beta=beta, snapshot_at=range(1, T + 1))
    for n in range(N):
        prev = S0[n]
        for t in range(T):
            decayed = np.exp(np.broadcast_to(lam[t, n], (dk,)))[:, None] * prev
            b = beta[t, n] * (v[t, n] - decayed.T @ k[t, n])
            np.testing.assert_allclose(res["b"][t, n], b, atol=1e-13)
            prev = res["snapshots"][t, n]


# ---------------------------------------------------------------------------------------------
# RWKV6: unrolled sum of outer products, bonus readout, Eq. 1 special case
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("T,dk,dv", [(1, 2, 2), (6, 4, 3), (8, 8, 4), (5, 2, 8)])
def test_rwkv6_matches_unrolled_sum_of_outer_products(T, dk, dv):
    N = 3
    S0, r, k, v, lam, _, bonus = rand_inputs(RWKV6, T, N, dk, dv)
    res = oracle.eager_rollout(RWKV6, S0, r, k, v, lam, bonus=bonus, snapshot_at=range(1, T + 1))
    w = np.exp(lam)

    def closed(n, t):  # S_t, t tokens consumed
        S = np.prod(w[:t, n], axis=0)[:, None] * S0[n] if t else S0[n].copy()
        for s in range(t):
            S = S + (np.prod(w[s + 1:t, n], axis=0) * k[s, n])[:, None] * v[s, n][None, :]
        return S

    for n in range(N):
        for t in range(1, T + 1):
            np.testing.assert_allclose(res["snapshots"][t - 1, n], closed(n, t), atol=1e-12)
            o = closed(n, t - 1).T @ r[t - 1, n] + np.dot(r[t - 1, n], bonus[n] * k[t - 1, n]) * v[t - 1, n]
            np.testing.assert_allclose(res["out"][t - 1, n], o, atol=1e-12)
        np.testing.assert_allclose(res["b"][:, n], v[:, n], atol=0)


def test_rwkv6_first_token_from_zero_state_is_pure_bonus():
    S0, r, k, v, lam, _, bonus = rand_inputs(RWKV6, 1, 2, 4, 3)
    res = oracle.eager_rollout(RWKV6, np.zeros_like(S0), r, k, v, lam, bonus=bonus)
    for n in range(2):
        np.testing.assert_allclose(res["out"][0, n], np.dot(r[0, n], bonus[n] * k[0, n]) * v[0, n], atol=1e-14)
        np.testing.assert_allclose(res["S"][n], np.outer(k[0, n], v[0, n]), atol=1e-14)


def test_rwkv6_without_decay_and_bonus_is_shifted_linear_attention():
    """w = 1, bonus = 0: S_t is the plain prefix sum of k v^T (Eq. 1) and o_t reads S_{t-1}."""
    T, N, dk, dv = 6, 2, 3, 4
    S0, r, k, v, lam, _, bonus = rand_inputs(RWKV6, T, N, dk, dv)
    res = oracle.eager_rollout(RWKV6, np.zeros_like(S0), r, k, v, np.zeros_like(lam),
                               bonus=np.zeros_like(bonus), snapshot_at=range(1, T + 1))
    for n in range(N):
        prefix = np.cumsum(np.einsum("tj,tc->tjc", k[:, n], v[:, n]), axis=0)
        np.testing.assert_allclose(res["snapshots"][:, n], prefix, atol=1e-13)
        np.testing.assert_allclose(res["out"][0, n], 0.0, atol=0)
        for t in range(1, T):
            np.testing.assert_allclose(res["out"][t, n], prefix[t - 1].T @ r[t, n], atol=1e-13)


# ---------------------------------------------------------------------------------------------
# invariants and special cases
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("op", [GDN, KDA])
def test_no_decay_no_write_keeps_state(op):
    T, N, dk, dv = 5, 2, 4, 4
    S0, q, k, v, lam, beta, _ = rand_inputs(op, T, N, dk, dv)
    res = oracle.eager_rollout(op, S0, q, k, v, np.zeros_like(lam), beta=np.zeros_like(beta), scale=2.0)
    np.testing.assert_allclose(res["S"], S0, atol=0)
    np.testing.assert_allclose(res["out"], 2.0 * np.einsum("njc,tnj->tnc", S0, q), atol=1e-13)
    np.testing.assert_allclose(res["b"], 0.0, atol=0)


def test_gdn_pure_scalar_decay_is_geometric():
    T, N, dk, dv = 7, 2, 3, 5
    S0, q, k, v, lam, beta, _ = rand_inputs(GDN, T, N, dk, dv)
    c = 0.8
    res = oracle.eager_rollout(GDN, S0, q, k, v, np.full_like(lam, np.log(c)), beta=np.zeros_like(beta),
                               snapshot_at=range(1, T + 1))
    for t in range(1, T + 1):
        np.testing.assert_allclose(res["snapshots"][t - 1], c ** t * S0, rtol=1e-13)


@pytest.mark.parametrize("op", [GDN, KDA])
def test_delta_rule_recall_with_unit_keys_and_full_write(op):
    """beta = 1 and ||k|| = 1: the updated state returns exactly v_t for key k_t, whatever the decay."""
    T, N, dk, dv = 6, 3, 8, 5
    S0, q, k, v, lam, beta, _ = rand_inputs(op, T, N, dk, dv, unit_keys=True)
    res = oracle.eager_rollout(op, S0, k.copy(), k, v, lam, beta=np.ones_like(beta))  # query with k itself
    np.testing.assert_allclose(res["out"], v, atol=1e-12)


def test_kda_with_equal_channels_is_gdn():
    T, N, dk, dv = 6, 2, 5, 4
    S0, q, k, v, lam, beta, _ = rand_inputs(GDN, T, N, dk, dv)
    a = oracle.eager_rollout(GDN, S0, q, k, v, lam, beta=beta)
    b = oracle.eager_rollout(KDA, S0, q, k, v, np.repeat(lam, dk, axis=-1), beta=beta)
    for key in ("out", "S", "b"):
        np.testing.assert_allclose(a[key], b[key], rtol=0, atol=1e-14)


@pytest.mark.parametrize("op", [GDN, KDA, RWKV6])
def test_superposition_in_state_and_values(op):
    T, N, dk, dv = 5, 2, 4, 3
    S0, q, k, v, lam, beta, bonus = rand_inputs(op, T, N, dk, dv)
    rng = np.random.default_rng(7)
    S0b, vb = rng.normal(size=S0.shape), rng.normal(size=v.shape)
    r1 = roll(op, S0, q, k, v, lam, beta, bonus)
    r2 = roll(op, S0b, q, k, vb, lam, beta, bonus)
    r3 = roll(op, 2 * S0 - 3 * S0b, q, k, 2 * v - 3 * vb, lam, beta, bonus)
    for key in ("out", "S"):
        np.testing.assert_allclose(r3[key], 2 * r1[key] - 3 * r2[key], atol=1e-11)


@pytest.mark.parametrize("op", [GDN, KDA])
def test_single_token_from_zero_state(op):
    S0, q, k, v, lam, beta, _ = rand_inputs(op, 1, 2, 4, 3)
    res = oracle.eager_rollout(op, np.zeros_like(S0), q, k, v, lam, beta=beta, scale=0.5)
    for n in range(2):
        np.testing.assert_allclose(res["S"][n], beta[0, n] * np.outer(k[0, n], v[0, n]), atol=1e-14)
        np.testing.assert_allclose(res["out"][0, n], 0.5 * beta[0, n] * np.dot(q[0, n], k[0, n]) * v[0, n], atol=1e-14)


def test_units_are_independent_and_rows_are_keys():
    """Swapping two units swaps their results; a decay on key channel 0 only touches state row 0."""
    T, N, dk, dv = 3, 2, 3, 4
    S0, q, k, v, lam, beta, bonus = rand_inputs(KDA, T, N, dk, dv)
    a = oracle.eager_rollout(KDA, S0, q, k, v, lam, beta=beta)
    b = oracle.eager_rollout(KDA, S0[::-1], q[:, ::-1], k[:, ::-1], v[:, ::-1], lam[:, ::-1], beta=beta[:, ::-1])
    np.testing.assert_allclose(a["out"], b["out"][:, ::-1], atol=0)
    lam1 = np.zeros((1, 1, dk)); lam1[0, 0, 0] = np.log(0.25)
    res = oracle.eager_rollout(KDA, S0[:1], q[:1, :1], k[:1, :1], v[:1, :1], lam1, beta=np.zeros((1, 1)))
    np.testing.assert_allclose(res["S"][0, 0], 0.25 * S0[0, 0], rtol=1e-15)
    np.testing.assert_allclose(res["S"][0, 1:], S0[0, 1:], atol=0)


def test_oracle_rejects_bad_arguments():
    S0, q, k, v, lam, beta, bonus = rand_inputs(GDN, 2, 1, 2, 2)
    with pytest.raises(ValueError):
        oracle.eager_rollout(GDN, S0, q, k, v, lam)            # beta missing
    with pytest.raises(ValueError):
        oracle.eager_rollout(RWKV6, S0, q, k, v, np.zeros((2, 1, 2)))  # bonus missing
    with pytest.raises(ValueError):
        oracle.eager_rollout(GDN, S0, q[:1], k, v, lam, beta=beta)     # ragged T
    with pytest.raises(ValueError):
        oracle.eager_rollout(GDN, S0, q, k, v, lam, beta=beta, snapshot_at=[2, 1])
    assert oracle.num_threads() >= 1


# ---------------------------------------------------------------------------------------------
# additive family (Table 1: linear attention, RetNet, GLA): the parallel (attention-matrix) form
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("op", [LINATTN, RETNET, GLA])
@pytest.mark.parametrize("T,dk,dv", [(1, 2, 3), (6, 4, 3), (9, 3, 5)])
def test_additive_family_matches_decay_masked_attention(op, T, dk, dv):
    """o_t = scale * [ (q_t . e^{L_t})^T S_0 + sum_{s<=t} ((q_t . e^{L_t - L_s}) . k_s) v_s ] with L the
    running sum of the log-decays (zero for linear attention, one scalar per head for RetNet): the
    masked-attention form these models are trained in; S_T likewise as a sum of decayed outer products."""
    N, scale = 2, 0.8
    S0, q, k, v, lam, _, _ = rand_inputs(op, T, N, dk, dv)
    res = roll(op, S0, q, k, v, lam, None, None, scale=scale)
    lam_full = np.broadcast_to(lam, (T, N, dk)) if lam.shape[-1] == 1 else lam
    Lc = np.cumsum(lam_full, axis=0)                                   # [T, N, dk]
    for n in range(N):
        for t in range(T):
            o = (q[t, n] * np.exp(Lc[t, n])) @ S0[n]
            for s_ in range(t + 1):
                o = o + np.dot(q[t, n] * np.exp(Lc[t, n] - Lc[s_, n]), k[s_, n]) * v[s_, n]
            np.testing.assert_allclose(res["out"][t, n], scale * o, atol=1e-12)
        S_T = np.exp(Lc[T - 1, n])[:, None] * S0[n]
        for s_ in range(T):
            S_T = S_T + np.outer(np.exp(Lc[T - 1, n] - Lc[s_, n]) * k[s_, n], v[s_, n])
        np.testing.assert_allclose(res["S"][n], S_T, atol=1e-12)
    np.testing.assert_array_equal(res["b"], v)


def test_additive_family_reductions():
    """GLA with equal channels is RetNet; RetNet with gamma = 1 is linear attention; linear attention
    from a zero state is the causal prefix sum of Eq. 1; RWKV6 with w = 1 and u = 1 reads the same
    state one token later."""
    T, N, dk, dv = 7, 2, 4, 3
    S0, q, k, v, lam1, _, _ = rand_inputs(RETNET, T, N, dk, dv)
    ret = oracle.eager_rollout(RETNET, S0, q, k, v, lam1, scale=1.1)
    gla = oracle.eager_rollout(GLA, S0, q, k, v, np.repeat(lam1, dk, axis=-1), scale=1.1)
    np.testing.assert_allclose(gla["out"], ret["out"], atol=1e-13)
    np.testing.assert_allclose(gla["S"], ret["S"], atol=1e-13)
    lin = oracle.eager_rollout(LINATTN, S0, q, k, v, None, scale=1.1)
    ret0 = oracle.eager_rollout(RETNET, S0, q, k, v, np.zeros_like(lam1), scale=1.1)
    np.testing.assert_allclose(lin["out"], ret0["out"], atol=1e-13)
    lin0 = oracle.eager_rollout(LINATTN, np.zeros_like(S0), q, k, v, None)
    prefix = np.cumsum(np.einsum("tnj,tnc->tnjc", k, v), axis=0)
    np.testing.assert_allclose(lin0["out"], np.einsum("tnjc,tnj->tnc", prefix, q), atol=1e-12)
    rw = oracle.eager_rollout(RWKV6, S0, q, k, v, np.zeros((T, N, dk)), bonus=np.ones((N, dk)))
    lin1 = oracle.eager_rollout(LINATTN, S0, q, k, v, None)
    np.testing.assert_allclose(rw["out"], lin1["out"], atol=1e-12)     # S_{t-1}^T r + (r.k) v = S_t^T r


# ---------------------------------------------------------------------------------------------
# base-plus-log schedule (Algorithm 1, Eq. 4-6): closure under append and merge
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("op", ALL_OPS)
@pytest.mark.parametrize("cap", [1, 2, 3, 5, 8])
def test_log_schedule_equals_eager_after_every_append_and_merge(op, cap):
    T, N, dk, dv = 11, 2, 4, 3
    S0, q, k, v, lam, beta, bonus = rand_inputs(op, T, N, dk, dv)
    ref = roll(op, S0, q, k, v, lam, beta, bonus, scale=1.3, snapshot_at=range(1, T + 1))
    st = logical.LogState(op, S0, cap)
    for t in range(T):
        if (st.length == cap).all():
            base_before = st.S_base.copy()
            logical.merge(st, only_if_full=True)
            assert (st.length == 0).all() and (st.lbar == 0).all()
            assert not np.array_equal(base_before, st.S_base)
            if t:  # the merge alone must not change the logical state
                np.testing.assert_allclose(logical.materialize(st), ref["snapshots"][t - 1], atol=1e-12)
        base_before = st.S_base.copy()
        out = logical.decode_step(st, q[t], k[t], v[t], lam[t], beta=beta[t], bonus=bonus, scale=1.3)
        np.testing.assert_array_equal(st.S_base, base_before)      # append never writes the base
        np.testing.assert_allclose(out, ref["out"][t], atol=1e-12)
        np.testing.assert_allclose(logical.materialize(st), ref["snapshots"][t], atol=1e-12)
        L = int(st.length[0])
        np.testing.assert_allclose(st.U_log[:, L - 1], ref["b"][t], atol=1e-12)   # U entry = b_t
        np.testing.assert_array_equal(st.K_log[:, L - 1], k[t])                    # K entry = a_t
        # the newest snapshot is the running cumulative decay, so lbar need not be stored separately
        np.testing.assert_array_equal(st.Lam_log[:, L - 1], st.lbar)
        first = t - (L - 1)
        np.testing.assert_allclose(st.Lam_log[:, L - 1], lam[first:t + 1].sum(axis=0).reshape(N, -1), atol=1e-13)


def test_log_schedule_merge_variants():
    op, cap, N, dk, dv = GDN, 4, 3, 3, 2
    S0, q, k, v, lam, beta, bonus = rand_inputs(op, 6, N, dk, dv)
    st = logical.LogState(op, S0, cap)
    logical.merge(st)                                   # empty log: identity
    np.testing.assert_array_equal(st.S_base, S0)
    for t in range(2):
        logical.decode_step(st, q[t], k[t], v[t], lam[t], beta=beta[t])
    logical.merge(st, only_if_full=True)                # not full: untouched
    assert (st.length == 2).all()
    np.testing.assert_array_equal(st.S_base, S0)
    full = logical.materialize(st)
    logical.merge(st)                                   # partial merge folds what is there
    assert (st.length == 0).all()
    np.testing.assert_allclose(st.S_base, full, atol=1e-14)
    for t in range(2, 6):
        logical.decode_step(st, q[t], k[t], v[t], lam[t], beta=beta[t])
    with pytest.raises(RuntimeError):
        logical.decode_step(st, q[0], k[0], v[0], lam[0], beta=beta[0])


@pytest.mark.parametrize("op", ALL_OPS)
@pytest.mark.parametrize("cap", [1, 3, 4])
def test_paper_cycle_with_fused_merge_step_equals_eager(op, cap):
    """The paper's own cycle: cap appends, then one step that consumes a token AND materialises
    (Algorithm 1, else-branch; Eq. 5 with the current-token term)."""
    T, N, dk, dv = 13, 2, 4, 3
    S0, q, k, v, lam, beta, bonus = rand_inputs(op, T, N, dk, dv)
    ref = roll(op, S0, q, k, v, lam, beta, bonus, scale=0.9, snapshot_at=range(1, T + 1))
    st = logical.LogState(op, S0, cap)
    for t in range(T):
        if (st.length == cap).all():
            out = logical.decode_merge_step(st, q[t], k[t], v[t], lam[t], beta=beta[t], bonus=bonus, scale=0.9)
            assert (st.length == 0).all() and (st.lbar == 0).all()
            np.testing.assert_allclose(st.S_base, ref["snapshots"][t], atol=1e-12)   # base alone is the state
        else:
            out = logical.decode_step(st, q[t], k[t], v[t], lam[t], beta=beta[t], bonus=bonus, scale=0.9)
        np.testing.assert_allclose(out, ref["out"][t], atol=1e-12)
        np.testing.assert_allclose(logical.materialize(st), ref["snapshots"][t], atol=1e-12)
    # on an empty log the fused step is the eager step
    st2 = logical.LogState(op, S0, cap)
    for t in range(3):
        out = logical.decode_merge_step(st2, q[t], k[t], v[t], lam[t], beta=beta[t], bonus=bonus, scale=0.9)
        np.testing.assert_allclose(out, ref["out"][t], atol=1e-12)
        np.testing.assert_allclose(st2.S_base, ref["snapshots"][t], atol=1e-12)


# ---------------------------------------------------------------------------------------------
# 16-bit (bfloat16) state: what is stored between tokens / between materialisations is rounded
# ---------------------------------------------------------------------------------------------
def test_bf16_rounding_is_round_to_nearest_even_and_matches_a_library_cast():
    torch = pytest.importorskip("torch")
    # hand-worked cases: bfloat16 keeps 8 significant bits, ulp(1.0) = 2^-7
    cases = {
        1.0: 1.0,
        1.0 + 2.0 ** -8: 1.0,                       # tie -> even mantissa (…0)
        1.0 + 3 * 2.0 ** -8: 1.0 + 2.0 ** -6,       # tie -> even mantissa (…10)
        1.0 + 2.0 ** -8 + 2.0 ** -20: 1.0 + 2.0 ** -7,   # just above the tie
        -(1.0 + 2.0 ** -8 + 2.0 ** -20): -(1.0 + 2.0 ** -7),
        0.0: 0.0,
        2.0 ** -20 * (1 + 2.0 ** -9): 2.0 ** -20,   # below half an ulp
        # fp64 -> fp32 comes first: 1 + 2^-8 + 2^-40 is a tie once it has been rounded to fp32
        1.0 + 2.0 ** -8 + 2.0 ** -40: 1.0,
    }
    for x, want in cases.items():
        assert float(logical.round_bf16(np.array([x]))[0]) == want, x
    x = np.concatenate([RNG.normal(0, 1, 4096), RNG.normal(0, 1e-3, 1024), RNG.normal(0, 300, 1024)])
    got = logical.round_bf16(x)
    want = torch.from_numpy(x).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(got, want)
    # exact ties on a grid: every odd multiple of half an ulp
    m = np.arange(129, 255, dtype=np.float64)
    ties = (2 * m + 1) * 2.0 ** -8 / 2
    want = torch.from_numpy(ties).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(logical.round_bf16(ties), want)
    assert logical.round_bf16(np.zeros((2, 3))).shape == (2, 3)


def test_eager_rollout_with_bf16_state_rounds_the_stored_state_after_every_token():
    torch = pytest.importorskip("torch")
    cast = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    # one token from a zero state, k = e_0, beta = 1, no decay: S_1[0, :] = v, so the stored row is cast(v)
    dk, dv = 3, 64
    v = RNG.normal(0, 1, (1, 1, dv))
    k = np.zeros((1, 1, dk)); k[0, 0, 0] = 1.0
    q = RNG.normal(0, 1, (1, 1, dk))
    r = oracle.eager_rollout(GDN, np.zeros((1, dk, dv)), q, k, v, np.zeros((1, 1, 1)), beta=np.ones((1, 1)),
                             state_bf16=True)
    np.testing.assert_array_equal(r["S"][0, 0], cast(v[0, 0]))
    np.testing.assert_array_equal(r["S"][0, 1:], 0.0)
    np.testing.assert_allclose(r["out"][0, 0], q[0, 0, 0] * v[0, 0], atol=1e-15)   # output: before the rounding
    # every operator: T tokens with rounding == T one-token rollouts, casting the state in between
    for op in ALL_OPS:
        T, N, dk, dv = 5, 2, 4, 3
        S0, q, k, v, lam, beta, bonus = rand_inputs(op, T, N, dk, dv)
        S0 = cast(S0)
        got = roll(op, S0, q, k, v, lam, beta, bonus, scale=1.1, snapshot_at=range(1, T + 1), state_bf16=True)
        S = S0
        for t in range(T):
            one = roll(op, S, q[t:t + 1], k[t:t + 1], v[t:t + 1], lam[t:t + 1], beta[t:t + 1], bonus, scale=1.1)
            np.testing.assert_allclose(got["out"][t], one["out"][0], atol=1e-13)
            S = cast(one["S"])
            np.testing.assert_array_equal(got["snapshots"][t], S)
        # and it is a different thing from the unrounded rollout
        plain = roll(op, S0, q, k, v, lam, beta, bonus, scale=1.1)
        assert np.max(np.abs(plain["S"] - got["S"])) > 1e-5


@pytest.mark.parametrize("op", ALL_OPS)
def test_log_schedule_with_bf16_base_rounds_once_per_materialisation(op):
    """Between materialisations nothing is rounded: with a representable S0 the logical state equals the
    exact eager recurrence; a merge (or the fused merge step) stores the rounded represented state."""
    torch = pytest.importorskip("torch")
    cast = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    T, N, dk, dv, cap = 9, 2, 4, 3, 4
    S0, q, k, v, lam, beta, bonus = rand_inputs(op, T, N, dk, dv)
    st = logical.LogState(op, S0, cap, store_base=logical.round_bf16)
    np.testing.assert_array_equal(st.S_base, cast(S0))             # the initial state is stored rounded
    S_start, t_start = st.S_base.copy(), 0
    for t in range(T):
        if (st.length == cap).all():
            if t == cap:      # first boundary: token-less merge
                exact = roll(op, S_start, q[t_start:t], k[t_start:t], v[t_start:t], lam[t_start:t],
                             beta[t_start:t], bonus)["S"]
                logical.merge(st)
                np.testing.assert_array_equal(st.S_base, cast(exact))
                S_start, t_start = st.S_base.copy(), t
            else:             # second boundary: the token is consumed by the merge step itself
                exact = roll(op, S_start, q[t_start:t + 1], k[t_start:t + 1], v[t_start:t + 1],
                             lam[t_start:t + 1], beta[t_start:t + 1], bonus)
                out = logical.decode_merge_step(st, q[t], k[t], v[t], lam[t], beta=beta[t], bonus=bonus)
                np.testing.assert_allclose(out, exact["out"][-1], atol=1e-12)   # output: unrounded state
                np.testing.assert_array_equal(st.S_base, cast(exact["S"]))
                S_start, t_start = st.S_base.copy(), t + 1
                continue
        out = logical.decode_step(st, q[t], k[t], v[t], lam[t], beta=beta[t], bonus=bonus)
        exact = roll(op, S_start, q[t_start:t + 1], k[t_start:t + 1], v[t_start:t + 1], lam[t_start:t + 1],
                     beta[t_start:t + 1], bonus)
        np.testing.assert_allclose(out, exact["out"][-1], atol=1e-12)
        np.testing.assert_allclose(logical.materialize(st), exact["S"], atol=1e-12)
    # capacity 1 through the merge step alone rounds after every token: the eager 16-bit-state recurrence
    st1 = logical.LogState(op, S0, 1, store_base=logical.round_bf16)
    ref = roll(op, cast(S0), q, k, v, lam, beta, bonus, snapshot_at=range(1, T + 1), state_bf16=True)
    for t in range(T):
        out = logical.decode_merge_step(st1, q[t], k[t], v[t], lam[t], beta=beta[t], bonus=bonus)
        np.testing.assert_allclose(out, ref["out"][t], atol=1e-12)
        np.testing.assert_array_equal(st1.S_base, ref["snapshots"][t])
