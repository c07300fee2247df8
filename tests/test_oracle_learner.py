"""Pins for the oracle's learner arithmetic (network, returns, A2C objective).

Each test checks the oracle against something fixed by the paper or by
mathematics alone: closed forms, finite differences, brute force written
independently here, special cases that reduce to a library routine.
"""
import os

import numpy as np
import pytest

from oracle import reference as R

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table2_hyperparameters.txt")


def golden():
    out = {}
    for line in open(GOLDEN):
        line = line.strip()
        if line and not line.startswith("#"):
            k, v = line.split()
            out[k] = float(v)
    return out


def test_defaults_match_table2():
    g = golden()
    hp = R.HParams()
    assert hp.lr == g["base_learning_rate"]
    assert hp.gamma == g["discount"]
    assert hp.ent_coef == g["entropy_coeff"]
    assert hp.vf_coef == g["vf_coeff"]
    assert hp.max_grad_norm == g["clip_global_gradient_norm"]
    net = R.Net.atari(6)
    assert (net.in_h, net.in_w, net.in_c) == (g["image_height"], g["image_width"], g["frame_stacking"])


def test_param_counts():
    # 3 conv + 1 hidden + heads at the measured sizes; MLP 8-64-64-(4+1)
    assert R.param_count(R.Net.mlp()) == 8 * 64 + 64 + 64 * 64 + 64 + 64 * 4 + 4 + 64 + 1 == 5061
    conv = 4 * 64 * 32 + 32 + 32 * 16 * 64 + 64 + 64 * 9 * 64 + 64 + 3136 * 512 + 512
    assert R.param_count(R.Net.atari(6)) == conv + 512 * 6 + 6 + 513 == 1687719
    assert R.param_count(R.Net.atari(18)) == conv + 512 * 18 + 18 + 513 == 1693875


# ------------------------------------------------------------------ returns
def test_returns_geometric_series():
    # constant reward, no episode ends: G_t = r (1-g^m)/(1-g) + g^m V_boot, m = T - t
    T, E, r, gam = 7, 3, 0.7, 0.9
    vb = np.array([2.0, -1.0, 0.5])
    G = R.returns(np.full((T, E), r), np.zeros((T, E), np.uint8), vb, gam)
    for t in range(T):
        m = T - t
        np.testing.assert_allclose(G[t], r * (1 - gam ** m) / (1 - gam) + gam ** m * vb, rtol=1e-13)


def test_returns_done_gamma0_and_one_step():
    rng = np.random.default_rng(0)
    T, E = 5, 4
    r = rng.normal(size=(T, E))
    vb = rng.normal(size=E)
    # gamma = 0: the return is the immediate reward
    np.testing.assert_array_equal(R.returns(r, np.zeros((T, E), np.uint8), vb, 0.0), r)
    # an episode end at step t cuts everything after it
    d = np.zeros((T, E), np.uint8)
    d[2, 1] = 1
    G = R.returns(r, d, vb, 0.99)
    assert G[2, 1] == r[2, 1]
    np.testing.assert_allclose(G[1, 1], r[1, 1] + 0.99 * r[2, 1], rtol=1e-15)
    # other environments are unaffected
    G0 = R.returns(r, np.zeros((T, E), np.uint8), vb, 0.99)
    np.testing.assert_array_equal(G[:, [0, 2, 3]], G0[:, [0, 2, 3]])
    # horizon 1: the one-step TD target
    G1 = R.returns(r[:1], np.zeros((1, E), np.uint8), vb, 0.99)
    np.testing.assert_allclose(G1[0], r[0] + 0.99 * vb, rtol=1e-15)


def test_returns_bruteforce_sum():
    # explicit sum_{i} gamma^i r_{t+i} prod(1-done) + bootstrap, written independently
    rng = np.random.default_rng(1)
    T, E, gam = 6, 5, 0.95
    r = rng.normal(size=(T, E))
    d = (rng.random((T, E)) < 0.25).astype(np.uint8)
    vb = rng.normal(size=E)
    G = R.returns(r, d, vb, gam)
    for e in range(E):
        for t in range(T):
            acc, alive, disc = 0.0, 1.0, 1.0
            for i in range(t, T):
                acc += disc * alive * r[i, e]
                alive *= 1.0 - d[i, e]
                disc *= gam
            acc += disc * alive * vb[e]
            assert abs(G[t, e] - acc) < 1e-12


# --------------------------------------------------------------------- loss
def _loss_value(z, a, adv, G, V, eta, cv):
    return R.a2c_loss(z, a, adv, G, V, eta, cv)[2][3]


def test_loss_uniform_policy():
    # uniform logits: pi = 1/A, entropy = log A, entropy gradient zero
    S, A = 5, 6
    z = np.full((S, A), 0.3)
    a = np.arange(S) % A
    adv = np.zeros(S)
    dz, dv, losses = R.a2c_loss(z, a, adv, np.zeros(S), np.zeros(S), 0.01, 0.5)
    assert abs(losses[2] - np.log(A)) < 1e-14
    assert np.abs(dz).max() < 1e-16
    # with advantages: -log pi(a) = log A
    adv = np.linspace(-1, 1, S)
    dz, dv, losses = R.a2c_loss(z, a, adv, np.zeros(S), np.zeros(S), 0.0, 0.5)
    assert abs(losses[0] - np.log(A) * adv.mean()) < 1e-14
    # dominant logit: entropy -> 0
    z2 = np.zeros((1, A)); z2[0, 2] = 60.0
    assert R.a2c_loss(z2, [2], [0.0], [0.0], [0.0], 0.01, 0.5)[2][2] < 1e-20


def test_loss_terms_and_signs():
    # hand-computed single sample, A = 2
    z = np.array([[np.log(3.0), 0.0]])  # pi = (3/4, 1/4)
    dz, dv, L = R.a2c_loss(z, [1], [2.0], [1.5], [0.5], 0.1, 0.5)
    H = -(0.75 * np.log(0.75) + 0.25 * np.log(0.25))
    assert abs(L[0] - (-np.log(0.25) * 2.0)) < 1e-14
    assert abs(L[1] - 1.0) < 1e-14          # (G - V)^2, no 1/2
    assert abs(L[2] - H) < 1e-14
    assert abs(L[3] - (L[0] - 0.1 * H + 0.5 * 1.0)) < 1e-14
    assert abs(dv[0] - 2 * 0.5 * (0.5 - 1.5)) < 1e-14
    # policy-gradient part: adv * (pi - onehot)
    dz0 = R.a2c_loss(z, [1], [2.0], [1.5], [0.5], 0.0, 0.5)[0]
    np.testing.assert_allclose(dz0[0], 2.0 * np.array([0.75, 0.25 - 1.0]), rtol=1e-14)


def test_loss_gradient_finite_difference():
    rng = np.random.default_rng(2)
    S, A = 7, 5
    z = rng.normal(size=(S, A)) * 2
    a = rng.integers(0, A, S)
    adv, G, V = rng.normal(size=S), rng.normal(size=S), rng.normal(size=S)
    dz, dv, _ = R.a2c_loss(z, a, adv, G, V, 0.03, 0.5)
    h = 1e-6
    for s in range(S):
        for k in range(A):
            zp, zm = z.copy(), z.copy()
            zp[s, k] += h; zm[s, k] -= h
            fd = (_loss_value(zp, a, adv, G, V, 0.03, 0.5) - _loss_value(zm, a, adv, G, V, 0.03, 0.5)) / (2 * h)
            assert abs(fd - dz[s, k]) < 1e-8
        Vp, Vm = V.copy(), V.copy()
        Vp[s] += h; Vm[s] -= h
        fd = (_loss_value(z, a, adv, G, Vp, 0.03, 0.5) - _loss_value(z, a, adv, G, Vm, 0.03, 0.5)) / (2 * h)
        assert abs(fd - dv[s]) < 1e-8
    # logits gradient of a softmax objective sums to zero over actions
    assert np.abs(dz.sum(axis=1)).max() < 1e-15


# ------------------------------------------------------------------ network
def _im2col_forward(net, params, obs):
    """Independent forward: convolutions lowered to matrix products (numpy),
    written here and nowhere in the oracle."""
    off = R.param_offsets(net)
    p = np.asarray(params, np.float64)
    x = np.asarray(obs, np.float64) * net.in_scale
    B = x.shape[0]
    x = x.reshape(B, net.in_h, net.in_w, net.in_c)
    f = (lambda t: np.maximum(t, 0)) if net.act == "relu" else np.tanh
    li = 0
    for (k, s, co) in net.convs:
        _, H, W, Cc = x.shape
        oh, ow = (H - k) // s + 1, (W - k) // s + 1
        cols = np.empty((B, oh, ow, k, k, Cc))
        for ky in range(k):
            for kx in range(k):
                cols[:, :, :, ky, kx, :] = x[:, ky:ky + s * oh:s, kx:kx + s * ow:s, :]
        Wm = p[off["L%d.W" % li]: off["L%d.W" % li] + co * k * k * Cc].reshape(co, k * k * Cc)
        b = p[off["L%d.b" % li]: off["L%d.b" % li] + co]
        x = f(cols.reshape(B, oh, ow, -1) @ Wm.T + b)
        li += 1
    x = x.reshape(B, -1)
    for h in net.hidden:
        Wm = p[off["L%d.W" % li]: off["L%d.W" % li] + h * x.shape[1]].reshape(h, x.shape[1])
        b = p[off["L%d.b" % li]: off["L%d.b" % li] + h]
        x = f(x @ Wm.T + b)
        li += 1
    H = x.shape[1]
    A = net.n_actions
    logits = x @ p[off["pi.W"]: off["pi.W"] + A * H].reshape(A, H).T + p[off["pi.b"]: off["pi.b"] + A]
    values = x @ p[off["v.W"]: off["v.W"] + H] + p[off["v.b"]]
    return logits, values


TINY_CONV = R.Net(6, 6, 2, ((3, 1, 3), (2, 2, 4)), (8,), "relu", 3, 0.5)
TINY_MLP = R.Net.mlp(5, 4, 3)


@pytest.mark.parametrize("net", [TINY_CONV, TINY_MLP, R.Net(9, 9, 3, ((3, 2, 5),), (6, 7), "tanh", 4, 1.0)])
def test_forward_matches_independent_lowering(net):
    rng = np.random.default_rng(3)
    p = rng.normal(size=R.param_count(net)) * 0.3
    obs = rng.normal(size=(4, net.in_size))
    z, v = R.forward(net, p, obs)
    z2, v2 = _im2col_forward(net, p, obs)
    np.testing.assert_allclose(z, z2, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(v, v2, rtol=1e-12, atol=1e-13)


def test_forward_full_size_layers_against_lowering():
    # the real 84x84x4 network on two frames, every trunk layer
    net = R.Net.atari(6)
    rng = np.random.default_rng(4)
    p = rng.normal(size=R.param_count(net)) * 0.02
    obs = rng.integers(0, 256, size=(2, net.in_size))
    z, v = R.forward(net, p, obs)
    z2, v2 = _im2col_forward(net, p, obs)
    np.testing.assert_allclose(z, z2, rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(v, v2, rtol=1e-10, atol=1e-12)
    assert R.forward(net, p, obs, which_layer=0)[2].shape == (2, 20, 20, 32)
    assert R.forward(net, p, obs, which_layer=2)[2].shape == (2, 7, 7, 64)


def test_conv_special_cases():
    # 1x1 kernel, stride 1: a per-pixel matrix product
    net = R.Net(4, 5, 3, ((1, 1, 2),), (3,), "relu", 2, 1.0)
    rng = np.random.default_rng(5)
    p = rng.normal(size=R.param_count(net))
    obs = rng.normal(size=(2, net.in_size))
    off = R.param_offsets(net)
    W = p[:6].reshape(2, 3)
    b = p[off["L0.b"]: off["L0.b"] + 2]
    y = R.forward(net, p, obs, which_layer=0)[2]
    np.testing.assert_allclose(y, np.maximum(obs.reshape(2, 4, 5, 3) @ W.T + b, 0), rtol=1e-13, atol=1e-14)
    # all-ones 2x2 kernel, zero bias, positive input: box sums
    net = R.Net(4, 4, 1, ((2, 1, 1),), (2,), "relu", 2, 1.0)
    p = np.zeros(R.param_count(net)); p[:4] = 1.0
    x = np.abs(rng.normal(size=(1, 4, 4, 1)))
    y = R.forward(net, p, x.reshape(1, -1), which_layer=0)[2]
    box = x[:, :-1, :-1] + x[:, 1:, :-1] + x[:, :-1, 1:] + x[:, 1:, 1:]
    np.testing.assert_allclose(y, box, rtol=1e-14)


def _objective(net, p, ro, hp):
    """The A2C objective with returns and advantages held constant (computed
    at the unperturbed parameters and passed in)."""
    obs = ro["obs"].reshape(-1, net.in_size)
    z, v = R.forward(net, p, obs)
    S = ro["S"]
    return R.a2c_loss(z[:S], ro["actions"].ravel(), ro["adv"], ro["G"], v[:S], hp.ent_coef, hp.vf_coef)[2][3]


@pytest.mark.parametrize("net", [TINY_CONV, TINY_MLP])
def test_learner_gradient_finite_difference(net):
    rng = np.random.default_rng(6)
    T, E = 3, 2
    hp = R.HParams(max_grad_norm=0.0, ent_coef=0.05)
    p = rng.normal(size=R.param_count(net)) * 0.4
    ro = dict(obs=rng.normal(size=(T + 1, E, net.in_size)),
              actions=rng.integers(0, net.n_actions, (T, E)).astype(np.int32),
              rewards=rng.normal(size=(T, E)).astype(np.float32),
              dones=(rng.random((T, E)) < 0.3).astype(np.uint8))
    info = R.learner_grad(net, p, ro, hp)
    ro.update(S=T * E, adv=info["adv"].ravel(), G=info["G"].ravel())
    g = info["grad"]
    h = 1e-6
    worst = 0.0
    for i in range(p.size):
        pp, pm = p.copy(), p.copy()
        pp[i] += h; pm[i] -= h
        fd = (_objective(net, pp, ro, hp) - _objective(net, pm, ro, hp)) / (2 * h)
        worst = max(worst, abs(fd - g[i]))
    # central differences in fp64: truncation O(h^2) + cancellation O(1e-16/h)
    assert worst < 1e-6 * np.abs(g).max(), (worst, np.abs(g).max())
    assert np.abs(g).min() > 0 or net.act == "relu"
    # advantage definition: A_t = G_t - V(s_t)
    np.testing.assert_array_equal(info["adv"], info["G"] - info["values"].reshape(T + 1, E)[:T])
    # chunked evaluation (used to spread the oracle over cores) is the same sum
    g2 = R.learner_grad(net, p, ro, hp, workers=3)["grad"]
    np.testing.assert_allclose(g2, g, rtol=1e-12, atol=1e-15)


def test_gradient_averaging_equals_bigger_batch():
    # n agents x b simulators, gradients averaged == one agent with n*b simulators
    # (footnote of Sec. 5 on A2C parallelised by all-reduce); pins the batch mean.
    net = TINY_MLP
    rng = np.random.default_rng(7)
    T, E, n = 3, 2, 3
    hp = R.HParams(max_grad_norm=0.0)
    p = rng.normal(size=R.param_count(net)) * 0.4
    ros = [dict(obs=rng.normal(size=(T + 1, E, net.in_size)),
                actions=rng.integers(0, net.n_actions, (T, E)).astype(np.int32),
                rewards=rng.normal(size=(T, E)), dones=np.zeros((T, E), np.uint8)) for _ in range(n)]
    gs = np.mean([R.learner_grad(net, p, r, hp)["grad"] for r in ros], axis=0)
    big = {k: np.concatenate([r[k] for r in ros], axis=1) for k in ros[0]}
    gb = R.learner_grad(net, p, big, hp)["grad"]
    np.testing.assert_allclose(gs, gb, rtol=1e-11, atol=1e-14)


# ----------------------------------------------------------------- sampling
def test_sampling_rule():
    z = np.log(np.array([[0.2, 0.5, 0.3]]))
    assert R.sample(z, [0.0])[0] == 0
    assert R.sample(z, [0.19999])[0] == 0
    assert R.sample(z, [0.2001])[0] == 1
    assert R.sample(z, [0.69])[0] == 1
    assert R.sample(z, [0.71])[0] == 2
    assert R.sample(z, [0.9999999])[0] == 2
    assert R.sample(z, [1.0])[0] == 2      # clamped
    rng = np.random.default_rng(8)
    n = 200000
    zz = np.repeat(z, n, axis=0)
    a = R.sample(zz, rng.random(n))
    freq = np.bincount(a, minlength=3) / n
    pi = np.array([0.2, 0.5, 0.3])
    assert np.all(np.abs(freq - pi) < 3 * np.sqrt(pi * (1 - pi) / n) + 1e-9)


# ------------------------------------------------- bf16-operand reading of "bf16 GEMMs"
def _bf16_independent(a):
    """bfloat16 rounding written independently: keep 8 significant bits, nearest, ties to even."""
    a = np.asarray(a, np.float64)
    out = np.zeros_like(a)
    nz = a != 0
    e = np.floor(np.log2(np.abs(a[nz])))
    q = 2.0 ** (e - 7)                       # spacing of bf16 numbers in [2^e, 2^(e+1))
    out[nz] = np.round(a[nz] / q) * q        # np.round: half to even
    return out


def test_bf16_rounding_rule():
    vals = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, 1.0 + 2 ** -9, -0.3, 255.0, 1e-3, 3.1415926, 0.0,
                     1.0 + 2 ** -8 + 2 ** -20, 129.5, 130.5])
    got = R.round_bf16(vals)
    np.testing.assert_array_equal(got, _bf16_independent(vals))
    assert got[1] == 1.0 and got[2] == 1.0 + 2 ** -6 and got[9] == 1.0 + 2 ** -7   # ties to even, above tie
    rng = np.random.default_rng(9)
    r = (rng.standard_normal(2000) * 10.0 ** rng.integers(-3, 3, 2000)).astype(np.float32).astype(np.float64)
    np.testing.assert_array_equal(R.round_bf16(r), _bf16_independent(r))


def test_bf16_operand_mode_is_exact_mode_on_rounded_operands():
    # One dense layer + heads, ReLU.  With bf16 operands the forward pass must equal the exact pass
    # run on weights rounded beforehand, followed by rounding of the stored activation.
    net = R.Net(1, 1, 6, (), (5,), "relu", 3, 1.0)
    rng = np.random.default_rng(10)
    p = rng.normal(size=R.param_count(net))
    obs = _bf16_independent(rng.normal(size=(4, 6)))
    off = R.param_offsets(net)
    pr = p.copy()
    pr[off["L0.W"]:off["L0.b"]] = _bf16_independent(p[off["L0.W"]:off["L0.b"]])
    h_exact = R.forward(net, pr, obs, which_layer=0)[2]
    z_b, v_b, h_b = R.forward(net.with_bf16(), p, obs, which_layer=0)
    np.testing.assert_array_equal(h_b, _bf16_independent(h_exact))
    W = p[off["pi.W"]:off["pi.b"]].reshape(3, 5)
    np.testing.assert_allclose(z_b, h_b @ W.T + p[off["pi.b"]:off["pi.b"] + 3], rtol=1e-14)
    # backward: gradient of the heads uses the rounded activation; the hidden layer's weight
    # gradient uses the rounded pre-activation gradient
    dz, dv = rng.normal(size=(4, 3)), rng.normal(size=4)
    g = R.backward(net.with_bf16(), p, obs, dz, dv)
    np.testing.assert_allclose(g[off["pi.W"]:off["pi.b"]].reshape(3, 5), dz.T @ h_b, rtol=1e-13)
    dh = (dz @ W + np.outer(dv, p[off["v.W"]:off["v.W"] + 5])) * (h_b > 0)
    dpre = _bf16_independent(dh)
    np.testing.assert_allclose(g[off["L0.W"]:off["L0.b"]].reshape(5, 6), dpre.T @ obs, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(g[off["L0.b"]:off["L0.b"] + 5], dpre.sum(axis=0), rtol=1e-13, atol=1e-15)


def test_bf16_operand_mode_stays_close_to_exact():
    rng = np.random.default_rng(11)
    net255 = R.Net(6, 6, 2, ((3, 1, 3), (2, 2, 4)), (8,), "relu", 3, 1.0 / 255.0)
    p = rng.normal(size=R.param_count(net255)) * 0.4
    obs = rng.integers(0, 256, size=(6, net255.in_size)).astype(np.float64)
    z, v = R.forward(net255, p, obs)
    zb, vb = R.forward(net255.with_bf16(), p, obs)
    assert np.linalg.norm(zb - z) <= 2e-2 * np.linalg.norm(z)
    assert np.linalg.norm(vb - v) <= 2e-2 * np.linalg.norm(v)


def test_float32_sum_variant_cancellation_and_bound():
    # The second evaluation of the rounded network (every trunk sum in float32, term after term) that the GPU
    # tests use to COUNT how many ReLU gates two valid implementations may disagree on.
    # (1) closed form: weights (2^30, 1, -2^30) on inputs (1, 1, 1), no bias.  Exactly the sum is 1 (gate open);
    #     in float32, 2^30 + 1 rounds to 2^30, so the running sum ends at 0 (gate closed).
    net = R.Net(1, 1, 3, (), (1,), "relu", 2, 1.0).with_bf16()
    p = np.zeros(R.param_count(net))
    off = R.param_offsets(net)
    p[off["L0.W"]:off["L0.W"] + 3] = [2.0 ** 30, 1.0, -2.0 ** 30]
    obs = np.ones((1, 3))
    assert R.forward(net, p, obs, which_layer=0)[2][0, 0] == 1.0
    assert R.forward(net.with_f32_sums(), p, obs, which_layer=0)[2][0, 0] == 0.0
    from tests.helpers import GATE_FAN_OUT, tie_allowance
    assert tie_allowance(net, p, obs) == 2 * GATE_FAN_OUT      # one gate disagrees (+ the one always granted)
    assert tie_allowance(net.with_bf16(False), p, obs) == 0     # the exact network has no such question
    # (2) on ordinary inputs the float32 sums stay within the textbook bound K u sum|w x| of the exact ones
    #     (u = 2^-24), and so do a conv layer's; the stored bf16 values then agree except for a few that sit on
    #     a rounding boundary, and no gate differs
    rng = np.random.default_rng(12)
    net2 = R.Net(6, 6, 2, ((3, 1, 4),), (16,), "relu", 3, 1.0)
    p2 = rng.normal(size=R.param_count(net2)) * 0.3
    o2 = rng.normal(size=(5, net2.in_size))
    for li, K in ((0, 18), (1, 64)):
        z = R.forward(net2, p2, o2, which_layer=li)[2]
        z32 = R.forward(net2.with_f32_sums(), p2, o2, which_layer=li)[2]
        scale = np.abs(z).max() * K
        assert np.abs(z32 - z).max() <= (K + 1) * 2.0 ** -24 * scale * 4
        assert np.abs(z32 - z).max() > 0                        # it really is another evaluation
    assert tie_allowance(net2.with_bf16(), p2, o2) == GATE_FAN_OUT
