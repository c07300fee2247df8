"""Pins for the oracle's optimiser and gossip arithmetic and its topology
schedules: closed forms, invariants of stochastic matrices, spectral facts
computed by brute force (dense matrices + SVD) on small agent counts.
"""
import os

import numpy as np
import pytest

from oracle import reference as R

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table2_hyperparameters.txt")


def _golden(key):
    for line in open(GOLDEN):
        if line.startswith(key + " "):
            return float(line.split()[1])
    raise KeyError(key)


# ------------------------------------------------------------------ RMSProp
def test_rmsprop_constant_gradient_closed_form():
    # v_0 = 0, constant gradient c: v_k = (1 - alpha^k) c^2
    alpha, lr, eps, c = 0.99, 7e-4, 1e-5, 0.3
    x, v = np.array([1.0, -2.0]), np.zeros(2)
    g = np.array([c, -c])
    for k in range(1, 6):
        x_prev = x
        x, v = R.rmsprop(x, g, v, 1.0, lr, alpha, eps)
        np.testing.assert_allclose(v, (1 - alpha ** k) * c * c, rtol=1e-13)
        np.testing.assert_allclose(x_prev - x, lr * g / (np.sqrt((1 - alpha ** k)) * c + eps), rtol=1e-12)
    # first step: lr * c / (sqrt(1-alpha)|c| + eps), sign follows the gradient
    y, _ = R.rmsprop([0.0], [c], [0.0], 1.0, lr, alpha, eps)
    assert abs(y[0] + lr * c / (np.sqrt(1 - alpha) * c + eps)) < 1e-18


def test_rmsprop_zero_gradient_and_clip_scaling():
    rng = np.random.default_rng(0)
    x, v = rng.normal(size=50), rng.random(50)
    y, v2 = R.rmsprop(x, np.zeros(50), v, 1.0, 7e-4, 0.99, 1e-5)
    np.testing.assert_array_equal(y, x)
    np.testing.assert_allclose(v2, 0.99 * v, rtol=1e-15)
    # clip coefficient c acts exactly like scaling the gradient
    g = rng.normal(size=50)
    ya, va = R.rmsprop(x, g, v, 0.25, 7e-4, 0.99, 1e-5)
    yb, vb = R.rmsprop(x, 0.25 * g, v, 1.0, 7e-4, 0.99, 1e-5)
    np.testing.assert_allclose(ya, yb, rtol=1e-15)
    np.testing.assert_allclose(va, vb, rtol=1e-15)
    # epsilon sits outside the root: with v -> 0 the step is lr*g/eps
    y, _ = R.rmsprop([0.0], [1e-12], [0.0], 1.0, 1.0, 1.0, 0.01)
    assert abs(y[0] + 1e-12 / 0.01) < 1e-22


def test_clip_coefficient():
    rng = np.random.default_rng(1)
    g = rng.normal(size=1000)
    mx = _golden("clip_global_gradient_norm")
    c, nrm = R.clip_coef(g, mx)
    assert abs(nrm - np.linalg.norm(g)) < 1e-12
    assert abs(np.linalg.norm(c * g) - min(nrm, mx)) < 1e-6
    small = g * (0.1 / nrm)
    assert R.clip_coef(small, mx)[0] == 1.0
    assert R.clip_coef(g, 0.0)[0] == 1.0     # off


# ----------------------------------------------------------------- topology
def test_ring_neighbours_and_weights():
    # directed ring v_1 -> v_2 -> ... -> v_n -> v_1: the in-peer of i is i-1
    n = 6
    for i in range(n):
        assert R.in_peers(R.RING, 1, n, 0, i) == [(i - 1) % n]
        assert R.in_peers(R.RING, 1, n, 17, i) == [(i - 1) % n]   # static graph
    P = R.mixing_matrix(R.RING, 1, n, 0)
    assert set(np.unique(P)) == {0.0, _golden("ring_mixing_weight")}
    S = np.roll(np.eye(n), -1, axis=1)        # S[i, i-1] = 1
    np.testing.assert_array_equal(P, (np.eye(n) + S) / 2)


@pytest.mark.parametrize("kind,peers", [(R.RING, 1), (R.RING, 2), (R.EXP, 1), (R.EXP, 2), (R.COMPLETE, 0)])
@pytest.mark.parametrize("n", [2, 3, 4, 7, 8, 32])
def test_matrices_are_doubly_stochastic(kind, peers, n):
    for k in range(7):
        P = R.mixing_matrix(kind, peers, n, k)
        assert (P >= 0).all()
        np.testing.assert_allclose(P.sum(axis=1), 1.0, atol=1e-15)   # row stochastic
        np.testing.assert_allclose(P.sum(axis=0), 1.0, atol=1e-15)   # columns too: mean preserved


def test_exponential_schedule_offsets():
    n = 8
    for k in range(6):
        for i in range(n):
            assert R.in_peers(R.EXP, 1, n, k, i) == [(i - 2 ** (k % 3)) % n]
            assert R.in_peers(R.EXP, 2, n, k, i) == [(i - 2 ** ((2 * k) % 3)) % n,
                                                     (i - 2 ** ((2 * k + 1) % 3)) % n]
    # non power of two: L = ceil(log2 n)
    assert R.in_peers(R.EXP, 1, 5, 2, 0) == [(0 - 4) % 5]
    assert R.in_peers(R.EXP, 1, 1, 0, 0) == []


@pytest.mark.parametrize("n", [4, 8, 16, 32, 64])
def test_exponential_graph_exact_consensus(n):
    # product of the log2(n) one-peer matrices is exactly 11^T / n
    L = n.bit_length() - 1
    M = np.eye(n)
    for k in range(L):
        M = R.mixing_matrix(R.EXP, 1, n, k) @ M
    np.testing.assert_allclose(M, np.full((n, n), 1.0 / n), atol=1e-15)


def test_two_peer_exponential_contraction_n32():
    M = np.eye(32)
    for k in range(5):
        M = R.mixing_matrix(R.EXP, 2, 32, k) @ M
    s = np.linalg.svd(M, compute_uv=False)
    assert abs(s[0] - 1.0) < 1e-12
    assert abs(s[1] - 1.0 / 9.0) < 1e-12


@pytest.mark.parametrize("n", [4, 8, 16])
def test_ring_second_singular_value(n):
    s = np.linalg.svd(R.mixing_matrix(R.RING, 1, n, 0), compute_uv=False)
    assert abs(s[1] - np.cos(np.pi / n)) < 1e-12


# ---------------------------------------------------------------------- mix
def test_mix_is_the_matrix_product():
    rng = np.random.default_rng(2)
    n, d = 8, 40
    Y = rng.normal(size=(n, d))
    for kind, peers in [(R.RING, 1), (R.EXP, 1), (R.EXP, 2), (R.COMPLETE, 0)]:
        for k in range(4):
            out = np.stack([R.mix(Y[i], [Y[j] for j in R.in_peers(kind, peers, n, k, i)]) for i in range(n)])
            np.testing.assert_allclose(out, R.mixing_matrix(kind, peers, n, k) @ Y, rtol=1e-13, atol=1e-15)


def test_mix_invariants():
    rng = np.random.default_rng(3)
    n, d = 8, 33
    hp = R.HParams(max_grad_norm=0.0)
    X = rng.normal(size=(n, d))
    Z = np.zeros((n, d))
    V = rng.random((n, d))
    for kind, peers in [(R.RING, 1), (R.EXP, 1), (R.EXP, 2)]:
        # zero gradients: pure gossip.  Column mean preserved, consensus distance contracts
        Xk = X
        for k in range(6):
            Xn, _, _ = R.sweep_sync(Xk, Z, V, hp, kind, peers, k)
            np.testing.assert_allclose(Xn.mean(axis=0), X.mean(axis=0), atol=1e-12)
            s2 = np.linalg.svd(R.mixing_matrix(kind, peers, n, k), compute_uv=False)[1]
            assert R.consensus_distance(Xn) <= s2 * R.consensus_distance(Xk) + 1e-12
            Xk = Xn
        # identical rows are a fixed point
        C = np.tile(X[:1], (n, 1))
        np.testing.assert_allclose(R.sweep_sync(C, Z, V, hp, kind, peers, 0)[0], C, rtol=1e-15)
    # ring: equality of the contraction on the first Fourier mode
    th = 2 * np.pi * np.arange(n) / n
    F = np.stack([np.cos(th), np.sin(th)], axis=1)
    Fn = R.sweep_sync(F, np.zeros_like(F), np.ones_like(F), hp, R.RING, 1, 0)[0]
    assert abs(R.consensus_distance(Fn) - np.cos(np.pi / n) * R.consensus_distance(F)) < 1e-12
    # exponential graph, n = 2^L: L rounds of pure gossip give the exact mean
    Xk = X
    for k in range(3):
        Xk = R.sweep_sync(Xk, Z, V, hp, R.EXP, 1, k)[0]
    np.testing.assert_allclose(Xk, np.tile(X.mean(axis=0), (n, 1)), atol=1e-14)


def test_sweep_sync_is_eq7():
    # X^(k+1) = P^(k) (X^(k) + dX^(k)) with dX the local optimiser step
    rng = np.random.default_rng(4)
    n, d = 4, 25
    hp = R.HParams(max_grad_norm=0.5)
    X, G, V = rng.normal(size=(n, d)), rng.normal(size=(n, d)), rng.random((n, d)) * 1e-2
    Xn, Vn, Y = R.sweep_sync(X, G, V, hp, R.RING, 1, 0)
    dX = np.empty_like(X)
    for i in range(n):
        c = min(1.0, 0.5 / (np.linalg.norm(G[i]) + 1e-6))
        v = 0.99 * V[i] + 0.01 * (c * G[i]) ** 2
        dX[i] = -7e-4 * c * G[i] / (np.sqrt(v) + 1e-5)
        np.testing.assert_allclose(Vn[i], v, rtol=1e-13)
    np.testing.assert_allclose(Y, X + dX, rtol=1e-13)
    np.testing.assert_allclose(Xn, R.mixing_matrix(R.RING, 1, n, 0) @ (X + dX), rtol=1e-13, atol=1e-16)


def test_replay_semantics():
    rng = np.random.default_rng(5)
    d = 20
    hp = R.HParams(max_grad_norm=0.0)
    x, g, v, m = rng.normal(size=d), rng.normal(size=d), rng.random(d), rng.normal(size=d)
    # no fresh message: the local update only (appendix, update without gossip)
    xn, vn, y = R.sweep_replay(x, g, v, hp, None)
    np.testing.assert_array_equal(xn, y)
    # fresh message: average of the updated parameters and the message
    xm, _, y2 = R.sweep_replay(x, g, v, hp, [m])
    np.testing.assert_array_equal(y2, y)
    np.testing.assert_allclose(xm, 0.5 * (y + m), rtol=1e-15)
    # no pending gradient: parameters and optimiser state untouched before mixing
    x0, v0, y0 = R.sweep_replay(x, None, v, hp, None)
    np.testing.assert_array_equal(x0, x); np.testing.assert_array_equal(v0, v)


def test_proposition1_bound():
    # identical initialisation, arbitrary update vectors:
    # ||X^(k+1) - mean|| <= sum_s beta^(k+1-s) ||dX^(s)||, beta = sigma_2 (ring: cos(pi/n))
    rng = np.random.default_rng(6)
    n, d = 8, 30
    hp = R.HParams(max_grad_norm=0.5)
    X = np.tile(rng.normal(size=(1, d)), (n, 1))
    V = np.zeros((n, d))
    beta = np.cos(np.pi / n)
    steps = []
    for k in range(12):
        G = rng.normal(size=(n, d)) * (1 + k % 3)
        Xn, V, Y = R.sweep_sync(X, G, V, hp, R.RING, 1, k)
        steps.append(np.linalg.norm(Y - X))      # ||alpha G^(k)||_F
        bound = sum(beta ** (k + 1 - s) * steps[s] for s in range(k + 1))
        assert R.consensus_distance(Xn) <= bound + 1e-12
        X = Xn


def test_prop1_bound_closed_forms():
    # constant step norm u and constant beta: a geometric series, u beta (1 - beta^(k+1)) / (1 - beta)
    u, beta, K = 0.37, 0.8, 9
    b = R.prop1_bound([u] * K, beta)
    for k in range(K):
        assert abs(b[k] - u * beta * (1 - beta ** (k + 1)) / (1 - beta)) < 1e-14
    # beta = 0: consensus after every round; beta = 1: the steps just add up
    steps = [0.5, 0.1, 2.0, 0.0, 0.3]
    np.testing.assert_array_equal(R.prop1_bound(steps, 0.0), np.zeros(5))
    np.testing.assert_allclose(R.prop1_bound(steps, 1.0), np.cumsum(steps), rtol=1e-15)
    # one factor per round: a round that averages exactly (factor 0) forgets everything before it
    b = R.prop1_bound([1.0, 2.0, 4.0], [0.5, 0.0, 0.25])
    np.testing.assert_allclose(b, [0.5, 0.0, 1.0], rtol=1e-15)


@pytest.mark.parametrize("kind,peers,n", [(R.EXP, 1, 8), (R.EXP, 2, 8), (R.RING, 2, 6)])
def test_prop1_bound_holds_with_per_round_factors(kind, peers, n):
    # the bound with every round's own contraction factor sigma_2(W_k) (brute force: SVD of the dense mixing
    # matrix) holds round by round and is never above the constant-beta bound with beta = max_k sigma_2(W_k)
    # (which is 1 for the exponential graphs: single rounds with shift n/2 do not contract every direction)
    rng = np.random.default_rng(11)
    d, K = 20, 9
    hp = R.HParams(max_grad_norm=0.5)
    X = np.tile(rng.normal(size=(1, d)), (n, 1))
    V = np.zeros((n, d))
    steps, s2 = [], []
    for k in range(K):
        G = rng.normal(size=(n, d)) * (0.0 if 3 <= k < 6 else 1.0 + k % 2)   # three pure-gossip rounds
        Xn, V, Y = R.sweep_sync(X, G, V, hp, kind, peers, k)
        steps.append(np.linalg.norm(Y - X))
        s2.append(np.linalg.svd(R.mixing_matrix(kind, peers, n, k), compute_uv=False)[1])
        b = R.prop1_bound(steps, s2)
        assert R.consensus_distance(Xn) <= b[k] * (1 + 1e-12) + 1e-12
        assert b[k] <= R.prop1_bound(steps, max(s2))[k] + 1e-12
        X = Xn
