"""CPU pins for the oracle's importance scores (Section 3.1: attention-layer score and Eq. 2)."""
import numpy as np
import pytest
from scipy.special import softmax

import oracle


def _ssm(seed, n_vis, M, H, G, n):
    r = np.random.default_rng(seed)
    T = n_vis + M
    return r.normal(size=(T, G, n)), r.normal(size=(T, G, n)), r.uniform(1e-3, 1e-1, size=(T, H))


def test_mamba_score_single_query_single_group_closed_form():
    B, C, dt = _ssm(0, 9, 1, 1, 1, 5)
    s = oracle.mamba_importance(B, C, dt, 9, 1)
    np.testing.assert_allclose(s, dt[:9, 0] * np.abs(B[:9, 0] @ C[9, 0]), rtol=1e-13)


def test_mamba_score_explicit_loops():
    n_vis, M, H, G, n = 7, 3, 6, 2, 4
    B, C, dt = _ssm(1, n_vis, M, H, G, n)
    s = oracle.mamba_importance(B, C, dt, n_vis, M)
    ref = np.zeros(n_vis)
    for i in range(n_vis):
        for g in range(G):
            dbar = sum(dt[i, h] for h in range(g * 3, g * 3 + 3)) / 3.0
            for m in range(M):
                ref[i] += abs(sum(dbar * B[i, g, k] * C[n_vis + m, g, k] for k in range(n)))
    np.testing.assert_allclose(s, ref / (M * G), rtol=1e-12)
    # equal to the per-head form normalised by 1/(M*H)
    per_head = np.zeros(n_vis)
    for h in range(H):
        g = h // 3
        per_head += (dt[:n_vis, h, None] * np.abs(B[:n_vis, g] @ C[n_vis:, g].T)).sum(axis=1)
    np.testing.assert_allclose(s, per_head / (M * H), rtol=1e-12)


def test_mamba_score_abs_is_inside_the_sum():
    # two queries c and -c: alignments cancel if summed before abs, double if abs first
    B, C, dt = _ssm(2, 5, 2, 2, 1, 4)
    C[6] = -C[5]
    s = oracle.mamba_importance(B, C, dt, 5, 2)
    one = oracle.mamba_importance(B[:6], C[:6], dt[:6], 5, 1)
    np.testing.assert_allclose(s, one, rtol=1e-13)
    assert np.all(s > 0)


def test_mamba_score_invariances():
    n_vis, M = 11, 4
    B, C, dt = _ssm(3, n_vis, M, 4, 2, 6)
    s = oracle.mamba_importance(B, C, dt, n_vis, M)
    perm = np.r_[np.arange(n_vis), n_vis + np.array([2, 0, 3, 1])]
    np.testing.assert_allclose(oracle.mamba_importance(B, C[perm], dt, n_vis, M), s, rtol=1e-13)
    np.testing.assert_allclose(oracle.mamba_importance(B, -2.5 * C, dt, n_vis, M), 2.5 * s, rtol=1e-13)
    # decay-free: A plays no role and visual C rows / text B rows are never read
    B2, C2 = B.copy(), C.copy()
    B2[n_vis:] = 99.0
    C2[:n_vis] = -77.0
    np.testing.assert_array_equal(oracle.mamba_importance(B2, C2, dt, n_vis, M), s)
    # visual-token order is respected
    vp = np.r_[np.arange(n_vis)[::-1], np.arange(n_vis, n_vis + M)]
    np.testing.assert_allclose(oracle.mamba_importance(B[vp], C[vp], dt[vp], n_vis, M), s[::-1], rtol=1e-13)


def test_mamba_score_orthogonal_query_scores_zero():
    B = np.zeros((3, 1, 2)); C = np.zeros((3, 1, 2))
    B[0, 0] = [1, 0]; B[1, 0] = [0, 2]; C[2, 0] = [0, 1]
    s = oracle.mamba_importance(B, C, np.full((3, 1), 0.5), 2, 1)
    np.testing.assert_allclose(s, [0.0, 1.0])


def _attn(seed, n_vis, M, Hq, Hkv, d):
    r = np.random.default_rng(seed)
    T = n_vis + M
    return r.normal(size=(T, Hq, d)), r.normal(size=(T, Hkv, d))


def test_attn_score_sums_to_one_and_uniform_for_zero_query():
    q, k = _attn(0, 13, 3, 4, 2, 8)
    s = oracle.attn_importance(q, k, 13, 3, 0.3)
    np.testing.assert_allclose(s.sum(), 1.0, rtol=1e-13)
    s0 = oracle.attn_importance(np.zeros_like(q), k, 13, 3, 0.3)
    np.testing.assert_allclose(s0, np.full(13, 1 / 13), rtol=1e-13)
    np.testing.assert_allclose(oracle.attn_importance(q[-4:], k[-4:], 1, 3, 0.3), [1.0], rtol=1e-13)


def test_attn_score_matches_library_softmax_and_gqa_mapping():
    n_vis, M, Hq, Hkv, d = 10, 4, 6, 2, 5
    q, k = _attn(1, n_vis, M, Hq, Hkv, d)
    scale = 1 / np.sqrt(d)
    s = oracle.attn_importance(q, k, n_vis, M, scale)
    kfull = np.repeat(k, Hq // Hkv, axis=1)                  # head h reads kv head h // 3
    logits = np.einsum("mhd,ihd->hmi", q[n_vis:], kfull[:n_vis]) * scale
    ref = softmax(logits, axis=2).sum(axis=(0, 1)) / (M * Hq)
    np.testing.assert_allclose(s, ref, rtol=1e-12)
    # text keys and visual queries are never read
    q2, k2 = q.copy(), k.copy()
    q2[:n_vis] = 50.0
    k2[n_vis:] = -50.0
    np.testing.assert_array_equal(oracle.attn_importance(q2, k2, n_vis, M, scale), s)


def test_attn_score_peaks_on_the_aligned_key():
    d = 4
    k = np.zeros((4, 1, d)); q = np.zeros((4, 1, d))
    k[1, 0, 0] = 1.0
    q[3, 0, 0] = 40.0
    s = oracle.attn_importance(q, k, 3, 1, 1.0)
    assert s.argmax() == 1 and s[1] > 0.999999


# ---- "Full Mamba Dynamic" score: |w_{t,i}| of Eq. 1, averaged over text positions and heads ----

def _ssm_dyn(seed, n_vis, M, H, G, n):
    B, C, dt = _ssm(seed, n_vis, M, H, G, n)
    A = -np.exp(np.random.default_rng(seed + 100).uniform(0.0, np.log(16.0), size=H))
    return B, C, dt, A


def test_full_dynamic_score_equals_unrolled_weights_of_eq1():
    # the pure-loop Eq. 1 weights (product of Abar written out factor by factor) of every head
    n_vis, M, H, G, n = 6, 3, 4, 2, 5
    B, C, dt, A = _ssm_dyn(20, n_vis, M, H, G, n)
    s = oracle.mamba_importance_full_dynamic(B, C, dt, A, n_vis, M)
    ref = np.zeros(n_vis)
    for h in range(H):
        w = oracle.mamba2_unrolled_weights(dt, A, B, C, h)          # [T, T], rows = output positions
        ref += np.abs(w[n_vis:, :n_vis]).sum(axis=0)
    np.testing.assert_allclose(s, ref / (M * H), rtol=1e-12)


def test_full_dynamic_score_is_the_response_of_the_recurrence_to_one_token():
    # w_{t,i} is what token i contributes to y_t: feed the sequential recurrence (the C loop) a one-hot x
    n_vis, M, H, G, n = 5, 2, 4, 2, 3
    B, C, dt, A = _ssm_dyn(21, n_vis, M, H, G, n)
    s = oracle.mamba_importance_full_dynamic(B, C, dt, A, n_vis, M)
    ref = np.zeros(n_vis)
    for i in range(n_vis):
        x = np.zeros((n_vis + M, H, 1))
        x[i] = 1.0
        y, _ = oracle.mamba2_recurrence(x, dt, A, B, C)
        ref[i] = np.abs(y[n_vis:, :, 0]).sum()
    np.testing.assert_allclose(s, ref / (M * H), rtol=1e-11)


def test_full_dynamic_score_without_decay_is_eq2():
    # A = 0 makes every Abar one: what is left is the content alignment, i.e. Eq. 2 (per-head form = group form)
    n_vis, M, H, G, n = 11, 4, 6, 3, 4
    B, C, dt, _ = _ssm_dyn(22, n_vis, M, H, G, n)
    s = oracle.mamba_importance_full_dynamic(B, C, dt, np.zeros(H), n_vis, M)
    np.testing.assert_allclose(s, oracle.mamba_importance(B, C, dt, n_vis, M), rtol=1e-12)


def test_full_dynamic_score_closed_form_constant_decay():
    # one head, one text row, dt = const: decay between token i and the text row is exp(A dt (n_vis - i))
    n_vis, n = 8, 3
    r = np.random.default_rng(23)
    B, C = r.normal(size=(n_vis + 1, 1, n)), r.normal(size=(n_vis + 1, 1, n))
    dt, A = np.full((n_vis + 1, 1), 0.25), np.array([-2.0])
    s = oracle.mamba_importance_full_dynamic(B, C, dt, A, n_vis, 1)
    i = np.arange(n_vis)
    ref = np.exp(-0.5 * (n_vis - i)) * 0.25 * np.abs(B[:n_vis, 0] @ C[n_vis, 0])
    np.testing.assert_allclose(s, ref, rtol=1e-13)


def test_full_dynamic_score_suppresses_early_tokens():
    # the paper's failure mode: with equal content alignment the score decays monotonically with distance
    n_vis, M, H = 40, 2, 2
    B = np.ones((n_vis + M, 1, 4)); C = np.ones((n_vis + M, 1, 4))
    dt = np.full((n_vis + M, H), 0.05); A = np.array([-1.0, -8.0])
    s = oracle.mamba_importance_full_dynamic(B, C, dt, A, n_vis, M)
    assert np.all(np.diff(s) > 0) and s[0] < 0.2 * s[-1]
    flat = oracle.mamba_importance(B, C, dt, n_vis, M)
    np.testing.assert_allclose(flat, flat[0], rtol=1e-13)            # Eq. 2 does not see position at all


# ---- attention score normalised by the model's own causal row (text keys m' <= m in the denominator) ----

def _attn(seed, n_vis, M, Hq, Hkv, d):
    r = np.random.default_rng(seed)
    return r.normal(size=(n_vis + M, Hq, d)), r.normal(size=(n_vis + M, Hkv, d))


def test_causal_row_attention_mass_is_what_the_attention_forward_applies():
    # one-hot values turn the attention output into the attention probabilities themselves
    n_vis, M, Hq, Hkv, d = 9, 4, 4, 2, 6
    q, k = _attn(30, n_vis, M, Hq, Hkv, d)
    T = n_vis + M
    P = np.zeros((T, Hq, T))                                        # P[t, h, j] = causal softmax of row t
    for c0 in range(0, T, d):                                       # d one-hot value columns per call
        cols = np.eye(T)[:, c0:c0 + d]
        v = np.zeros((T, Hkv, d)); v[:, :, :cols.shape[1]] = cols[:, None, :]
        P[:, :, c0:c0 + cols.shape[1]] = oracle.attention_forward(q, k, v, 0.3)[:, :, :cols.shape[1]]
    np.testing.assert_allclose(P.sum(axis=2), 1.0, rtol=1e-12)
    ref = P[n_vis:, :, :n_vis].sum(axis=(0, 1)) / (M * Hq)
    np.testing.assert_allclose(oracle.attn_importance(q, k, n_vis, M, 0.3, "causal_row"), ref, rtol=1e-12)


def test_causal_row_attention_mass_closed_forms():
    n_vis, M, Hq, Hkv, d = 7, 3, 2, 1, 4
    q, k = _attn(31, n_vis, M, Hq, Hkv, d)
    # zero queries: every causal row is uniform over its n_vis + m + 1 keys
    s = oracle.attn_importance(np.zeros_like(q), k, n_vis, M, 1.0, "causal_row")
    np.testing.assert_allclose(s, np.mean([1.0 / (n_vis + m + 1) for m in range(M)]), rtol=1e-13)
    # the two normalisations differ by the share of each row's mass that stays on visual keys
    sv = oracle.attn_importance(q, k, n_vis, M, 0.5)
    sc = oracle.attn_importance(q, k, n_vis, M, 0.5, "causal_row")
    assert abs(sv.sum() - 1.0) < 1e-12 and 0.0 < sc.sum() < 1.0 and np.all(sc < sv)
    # a text key is invisible to earlier text queries: make the LAST text key overwhelmingly attractive; the
    # first M-1 queries must keep all their visual mass (what is left over is the last query's share, >= 0)
    k2 = k.copy(); k2[-1] = 50.0 * np.sign(q[n_vis:].mean(axis=(0, 1)))[None, :]
    sc2 = oracle.attn_importance(q, k2, n_vis, M, 0.5, "causal_row")
    first = oracle.attn_importance(q[:-1], k[:-1], n_vis, M - 1, 0.5, "causal_row") * (M - 1)
    last_share = sc2 * M - first
    assert np.all(last_share >= -1e-12) and last_share.sum() <= 1.0 + 1e-12
