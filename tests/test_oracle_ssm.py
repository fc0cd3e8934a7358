"""CPU pins for the oracle's Mamba-2 recurrence (Section 3.1 and the appendix derivation).

The recurrence is checked against things fixed by the paper and by mathematics, not against
itself: the unrolled weighted sum (Eq. 1), a geometric-series closed form, the zero-decay limit
(causal linear attention through a library matmul), the strong-decay limit, linearity in the
initial state, and the head-to-group mapping.
"""
import numpy as np
import pytest

import oracle


def _rand(seed, T, H, p, n, G, dt_scale=1.0):
    r = np.random.default_rng(seed)
    x = r.normal(size=(T, H, p))
    dt = r.uniform(1e-3, 1e-1, size=(T, H)) * dt_scale
    A = -np.exp(r.uniform(0, np.log(16), size=H))
    B = r.normal(size=(T, G, n))
    C = r.normal(size=(T, G, n))
    return x, dt, A, B, C


@pytest.mark.parametrize("shape", [(1, 1, 1, 1, 1), (9, 2, 3, 5, 1), (33, 4, 3, 5, 2), (40, 6, 2, 7, 3)])
def test_recurrence_equals_unrolled_sum(shape):
    x, dt, A, B, C = _rand(1, *shape, dt_scale=5.0)
    y, _ = oracle.mamba2_recurrence(x, dt, A, B, C)
    np.testing.assert_allclose(y, oracle.mamba2_unrolled(x, dt, A, B, C), rtol=1e-11, atol=1e-12)


def test_geometric_series_closed_form():
    # p=n=1, x=b=c=1, constant dt: y_t = dt * (1 - r^(t+1)) / (1 - r), r = exp(dt*A)
    T, delta, a = 50, 0.07, -3.0
    one = np.ones((T, 1, 1))
    y, S = oracle.mamba2_recurrence(one, np.full((T, 1), delta), np.array([a]), one, one)
    r = np.exp(delta * a)
    t = np.arange(T)
    np.testing.assert_allclose(y[:, 0, 0], delta * (1 - r ** (t + 1)) / (1 - r), rtol=1e-12)
    np.testing.assert_allclose(S[0, 0, 0], y[-1, 0, 0], rtol=1e-12)
    w = oracle.mamba2_unrolled_weights(np.full((T, 1), delta), np.array([a]), one, one, 0)
    np.testing.assert_allclose(w[T - 1], delta * r ** (T - 1 - t), rtol=1e-12)
    assert np.all(np.triu(w, 1) == 0)


def test_one_token_closed_form():
    x, dt, A, B, C = _rand(2, 1, 3, 4, 6, 1)
    y, S = oracle.mamba2_recurrence(x, dt, A, B, C)
    for h in range(3):
        np.testing.assert_allclose(y[0, h], dt[0, h] * np.dot(B[0, 0], C[0, 0]) * x[0, h], rtol=1e-12)
        np.testing.assert_allclose(S[h], np.outer(x[0, h], dt[0, h] * B[0, 0]), rtol=1e-12)


def test_zero_decay_is_causal_linear_attention():
    T, H, p, n, G = 24, 2, 3, 4, 1
    x, dt, A, B, C = _rand(3, T, H, p, n, G)
    y, _ = oracle.mamba2_recurrence(x, dt, np.zeros(H), B, C)
    for h in range(H):
        ref = np.tril(C[:, 0] @ B[:, 0].T) @ (dt[:, h, None] * x[:, h])
        np.testing.assert_allclose(y[:, h], ref, rtol=1e-11, atol=1e-12)


def test_strong_decay_keeps_only_current_token():
    T, H, p, n, G = 12, 2, 3, 4, 2
    x, dt, A, B, C = _rand(4, T, H, p, n, G)
    y, _ = oracle.mamba2_recurrence(x, dt, np.full(H, -1e5), B, C)
    for h in range(H):
        ref = (dt[:, h] * np.einsum("tk,tk->t", B[:, h], C[:, h]))[:, None] * x[:, h]
        np.testing.assert_allclose(y[:, h], ref, rtol=1e-9, atol=1e-12)


def test_initial_state_and_skip_term():
    T, H, p, n, G = 10, 2, 3, 4, 1
    x, dt, A, B, C = _rand(5, T, H, p, n, G)
    r = np.random.default_rng(6)
    S0, D = r.normal(size=(H, p, n)), r.normal(size=H)
    y0, _ = oracle.mamba2_recurrence(x, dt, A, B, C)
    y1, _ = oracle.mamba2_recurrence(x, dt, A, B, C, D=D, init_state=S0)
    for h in range(H):
        carry = np.exp(np.cumsum(dt[:, h] * A[h]))[:, None] * (C[:, 0] @ S0[h].T)
        np.testing.assert_allclose(y1[:, h] - y0[:, h], carry + D[h] * x[:, h], rtol=1e-10, atol=1e-12)
    # splitting the sequence and carrying the state reproduces the full run
    ya, Sa = oracle.mamba2_recurrence(x[:4], dt[:4], A, B[:4], C[:4])
    yb, _ = oracle.mamba2_recurrence(x[4:], dt[4:], A, B[4:], C[4:], init_state=Sa)
    np.testing.assert_allclose(np.concatenate([ya, yb]), y0, rtol=1e-12, atol=1e-13)


def test_heads_read_their_own_group():
    T, H, p, n, G = 8, 4, 2, 3, 2
    x, dt, A, B, C = _rand(7, T, H, p, n, G)
    y, _ = oracle.mamba2_recurrence(x, dt, A, B, C)
    B2 = B.copy()
    B2[:, 1] += 1.0                                   # touch group 1 only
    y2, _ = oracle.mamba2_recurrence(x, dt, A, B2, C)
    assert np.array_equal(y[:, :2], y2[:, :2]) and not np.allclose(y[:, 2:], y2[:, 2:])


@pytest.mark.parametrize("Q", [1, 3, 8, 16, 37, 64, 100])
def test_chunked_equals_sequential(Q):
    x, dt, A, B, C = _rand(8, 37, 4, 3, 5, 2, dt_scale=3.0)
    y, S = oracle.mamba2_recurrence(x, dt, A, B, C)
    yc, Sc = oracle.mamba2_chunked(x, dt, A, B, C, Q)
    np.testing.assert_allclose(yc, y, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(Sc, S, rtol=1e-11, atol=1e-12)


def test_chunked_survives_large_cumulative_decay():
    # cumulative log-decay far below the fp64 underflow of exp(l)*exp(-l) factorisations
    T = 600
    x, dt, A, B, C = _rand(9, T, 1, 2, 3, 1)
    dt[:] = 0.1
    A[:] = -16.0
    y, _ = oracle.mamba2_recurrence(x, dt, A, B, C)
    yc, _ = oracle.mamba2_chunked(x, dt, A, B, C, 512)
    assert np.all(np.isfinite(yc))
    np.testing.assert_allclose(yc, y, rtol=1e-10, atol=1e-12)
