"""Pins of the oracle's attention on the representative set (Section 2.3, Eq. 2).

The function is the definition written out; what fixes it from outside: softmax rows sum to
one (constant values pass through), the case r = T is ordinary dense attention (stated here
independently with numpy), a single representative returns its own value row, a brute-force
pure-Python evaluation on a tiny input, invariance of softmax under a per-row shift of the
scores, and the expansion rule of Section 2.3 (a redundant token takes its nearest
representative's output).
"""
import math

import numpy as np
import pytest

import oracle


def rand_qkv(T, h, d_h, seed):
    rng = np.random.default_rng(seed)
    return tuple(rng.standard_normal((T, h, d_h)) for _ in range(3))


def dense_attention_numpy(Q, K, V, causal=False):
    """softmax(Q K^T / sqrt(d_h)) V per head, with numpy matrix products."""
    T, h, d_h = Q.shape
    out = np.empty_like(Q)
    for j in range(h):
        S = Q[:, j, :] @ K[:, j, :].T / math.sqrt(d_h)
        if causal:
            S = np.where(np.tril(np.ones((T, T), dtype=bool)), S, -np.inf)
        S = S - S.max(axis=1, keepdims=True)
        P = np.exp(S)
        P /= P.sum(axis=1, keepdims=True)
        out[:, j, :] = P @ V[:, j, :]
    return out


@pytest.mark.parametrize("causal", [False, True])
def test_all_tokens_representative_is_dense_attention(causal):
    Q, K, V = rand_qkv(37, 3, 16, 1)
    got = oracle.attention_reps(Q, K, V, np.arange(37), causal=causal)
    assert np.max(np.abs(got - dense_attention_numpy(Q, K, V, causal))) < 1e-12


def test_restriction_to_the_representative_rows():
    """Eq. 2 on R equals dense attention of the sub-matrices Q_R, K_R, V_R; other rows stay 0."""
    Q, K, V = rand_qkv(50, 2, 8, 2)
    R = np.array([0, 3, 4, 17, 30, 49])
    got = oracle.attention_reps(Q, K, V, R)
    ref = dense_attention_numpy(Q[R], K[R], V[R])
    assert np.max(np.abs(got[R] - ref)) < 1e-12
    rest = np.setdiff1d(np.arange(50), R)
    assert np.all(got[rest] == 0.0)


def test_softmax_rows_sum_to_one():
    Q, K, V = rand_qkv(40, 2, 8, 3)
    V[:] = 1.0
    R = np.arange(0, 40, 3)
    got = oracle.attention_reps(Q, K, V, R)
    assert np.max(np.abs(got[R] - 1.0)) < 1e-13


def test_single_representative_returns_its_value_row():
    Q, K, V = rand_qkv(20, 4, 8, 4)
    near = np.full(20, 7, dtype=np.int32)
    got = oracle.attention_reps(Q, K, V, [7], nearest_idx=near)
    assert np.max(np.abs(got - V[7][None])) < 1e-15      # every token takes V[7]


def test_causal_first_representative_sees_only_itself():
    Q, K, V = rand_qkv(30, 2, 8, 5)
    R = np.array([2, 9, 21])
    got = oracle.attention_reps(Q, K, V, R, causal=True)
    assert np.max(np.abs(got[2] - V[2])) < 1e-15


def test_brute_force_tiny():
    Q, K, V = rand_qkv(6, 1, 2, 6)
    R = [1, 2, 5]
    got = oracle.attention_reps(Q, K, V, R)
    for i in R:
        w = [math.exp(sum(Q[i, 0, c] * K[k, 0, c] for c in range(2)) / math.sqrt(2)) for k in R]
        z = sum(w)
        for c in range(2):
            assert abs(got[i, 0, c] - sum(w[n] / z * V[k, 0, c] for n, k in enumerate(R))) < 1e-12


def test_scaling_uses_sqrt_of_head_width():
    """One query against two keys with known scores: the weights are exp(s/sqrt(d_h))."""
    d_h = 16
    Q = np.zeros((2, 1, d_h)); K = np.zeros((2, 1, d_h)); V = np.zeros((2, 1, d_h))
    Q[0, 0, 0] = 4.0
    K[0, 0, 0], K[1, 0, 0] = 1.0, 3.0                    # scores 4 and 12 -> /4 -> 1 and 3
    V[0, 0, 0], V[1, 0, 0] = 1.0, -1.0
    got = oracle.attention_reps(Q, K, V, [0, 1])
    w0, w1 = math.exp(1.0), math.exp(3.0)
    assert abs(got[0, 0, 0] - (w0 - w1) / (w0 + w1)) < 1e-14


def test_softmax_shift_invariance_and_expansion():
    Q, K, V = rand_qkv(25, 2, 8, 7)
    R = np.array([0, 5, 6, 11, 20])
    a = oracle.attention_reps(Q, K, V, R)
    # adding the same vector u to every key shifts row i's scores by the constant q_i . u, which
    # softmax ignores
    u = np.random.default_rng(8).standard_normal((1, 2, 8))
    b = oracle.attention_reps(Q, K + u, V, R)
    assert np.max(np.abs(a - b)) < 1e-12
    # expansion: token t takes the output of nearest[t]; representatives map to themselves
    near = np.array([R[(t * 3) % R.size] for t in range(25)], dtype=np.int32)
    near[R] = R
    e = oracle.attention_reps(Q, K, V, R, nearest_idx=near)
    for t in range(25):
        assert np.array_equal(e[t], a[near[t]])
    near[3] = -1                                         # no representative: row left at zero
    e = oracle.attention_reps(Q, K, V, R, nearest_idx=near)
    assert np.all(e[3] == 0.0)
