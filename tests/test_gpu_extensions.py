"""GPU parity of the pieces beyond the core step: the staleness bound of Sec. 3, the distance
from consensus of Propositions 1-2, and the gradient all-reduce of the synchronous A2C baseline."""
import numpy as np
import pytest

import gala_inputs as GI
from oracle import reference as R
from tests.helpers import TOL_FP32_NET, TOL_SWEEP, assert_close, oracle_hp, oracle_net

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def _learner(w, **hp):
    from paper_1906_04585_b200 import learner as LM
    return LM.Learner(w.n_agents, w.topo_kind, w.topo_peers, w.net_kind, w.n_actions, w.n_envs, w.n_steps,
                      obs_dim=w.obs_dim, hidden=w.hidden, **hp)


def test_consensus_distance_matches_oracle_and_contracts():
    from paper_1906_04585_b200 import binding as B
    w = GI.WORKLOADS[0].scaled(n_agents=8, topo_kind=R.EXP)
    L = _learner(w, max_grad_norm=0.0)
    rng = np.random.default_rng(5)
    X = rng.normal(size=(w.n_agents, L.d)).astype(np.float32) * 0.1
    for i in range(w.n_agents):
        L.set_state(i, params=X[i], sq_avg=np.zeros(L.d, np.float32))
    d0 = B.gala_consensus_distance(L.ctx)
    assert abs(d0 - R.consensus_distance(X)) <= 1e-9 * d0
    # pure gossip (zero gradients): each round contracts by at most sigma_2 of that round's matrix, and
    # log2(8) rounds of the 1-peer exponential graph reach the mean exactly (up to fp32 rounding)
    prev = d0
    for k in range(3):
        for i in range(w.n_agents):
            L.set_grad(i, np.zeros(L.d, np.float32), 1.0)
        L.step_sync(None)
        dk = B.gala_consensus_distance(L.ctx)
        s2 = np.linalg.svd(R.mixing_matrix(R.EXP, 1, w.n_agents, k), compute_uv=False)[1]
        assert dk <= s2 * prev * (1 + 1e-5) + 1e-6
        prev = dk
    assert prev <= 1e-5 * d0
    Xn = np.stack([L.get_params(i) for i in range(w.n_agents)])
    assert_close("mean", Xn[3], X.astype(np.float64).mean(axis=0), 1e-5)
    L.close()


def test_allreduce_a2c_mode_matches_oracle():
    # complete graph: gradients averaged over agents, the average clipped, one common RMSProp step
    w = GI.WORKLOADS[0].scaled(n_agents=5, topo_kind=R.COMPLETE, topo_peers=0)
    net = oracle_net(w)
    L = _learner(w)
    ohp = oracle_hp(L.hp)
    from paper_1906_04585_b200 import learner as LM
    p0 = GI.init_params(GI.net_tensors(w), w.seed)
    for i in range(w.n_agents):
        L.set_state(i, params=p0, sq_avg=np.zeros(L.d, np.float32))
    X = p0.astype(np.float64)
    V = np.zeros_like(X)
    for k in range(2):
        ros = [GI.rollout(w, i, k) for i in range(w.n_agents)]
        dev = [LM.DeviceRollout(r) for r in ros]
        L.step_sync(dev)
        L.sync()
        gm = np.mean([R.learner_grad(net, X, r, ohp)["grad"] for r in ros], axis=0)
        # the same as one agent with all simulators (footnote of Sec. 5)
        big = {key: np.concatenate([r[key] for r in ros], axis=1) for key in ros[0]}
        np.testing.assert_allclose(gm, R.learner_grad(net, X, big, ohp)["grad"], rtol=1e-9, atol=1e-14)
        c, _ = R.clip_coef(gm, ohp.max_grad_norm)
        X, V = R.rmsprop(X, gm, V, c, ohp.lr, ohp.rms_alpha, ohp.rms_eps)
        for i in range(w.n_agents):
            assert_close("g[%d]" % i, L.get_grad(i), gm, TOL_FP32_NET)
            assert_close("x[%d]" % i, L.get_params(i), X, TOL_SWEEP)
            assert_close("v[%d]" % i, L.get_sq_avg(i), V, 2 * TOL_FP32_NET)
    from paper_1906_04585_b200 import binding as B
    assert B.gala_consensus_distance(L.ctx) < 1e-6        # all agents stay identical
    with pytest.raises(B.GalaError):
        L.gossip(0)
    L.close()


def test_allreduce_a2c_mode_conv_net_matches_oracle():
    # the same mode on the conv net (the path the benchmark's all-reduce leg times): the gradient every agent
    # holds after the round is the oracle's mean over agents (footnote of Sec. 5: one agent with all simulators),
    # per element; the common RMSProp step is replayed from that gradient and its norm at the tolerance of the pass
    from paper_1906_04585_b200 import binding as B
    from paper_1906_04585_b200 import learner as LM
    from tests.helpers import TOL_BF16, assert_grad_close, tie_allowance
    w = GI.WORKLOADS[1].scaled(n_agents=2, n_envs=3, n_steps=2, topo_kind=R.COMPLETE, topo_peers=0)
    net = oracle_net(w)
    L = _learner(w)
    ohp = oracle_hp(L.hp)
    p0 = GI.init_params(GI.net_tensors(w), w.seed)
    for i in range(w.n_agents):
        L.set_state(i, params=p0, sq_avg=np.zeros(L.d, np.float32))
    X = p0.astype(np.float64)
    ros = [GI.rollout(w, i, 0) for i in range(w.n_agents)]
    L.step_sync([LM.DeviceRollout(r) for r in ros])
    L.sync()
    gm = np.mean([R.learner_grad(net, X, r, ohp)["grad"] for r in ros], axis=0)
    big = {key: np.concatenate([r[key] for r in ros], axis=1) for key in ros[0]}
    g_big = R.learner_grad(net, X, big, ohp)["grad"]
    assert np.linalg.norm(gm - g_big) <= 1e-9 * np.linalg.norm(g_big)
    S = w.n_envs * w.n_steps
    allow = sum(tie_allowance(net, X, r["obs"].reshape(-1, 84 * 84 * 4)[:S]) for r in ros)
    g0 = L.get_grad(0)
    assert_grad_close("mean gradient", g0, gm, net, TOL_BF16, max_outliers=allow)
    nrm = float(np.float32(B.gala_losses(L.ctx, 0)[3]))
    assert abs(nrm - np.linalg.norm(gm)) <= TOL_BF16 * np.linalg.norm(gm)
    c = min(1.0, ohp.max_grad_norm / (nrm + 1e-6))
    xn, vn = R.rmsprop(X, g0.astype(np.float64), np.zeros_like(X), c, ohp.lr, ohp.rms_alpha, ohp.rms_eps)
    for i in range(w.n_agents):
        np.testing.assert_array_equal(L.get_grad(i), g0)              # every agent holds the same mean
        assert_close("x[%d]" % i, L.get_params(i), xn, TOL_SWEEP)
        assert_close("v[%d]" % i, L.get_sq_avg(i), vn, TOL_SWEEP)
    assert B.gala_consensus_distance(L.ctx) == 0.0
    L.close()


def test_update_norm_matches_oracle_and_proposition1_bound_holds():
    # Identical initial parameters, real rollouts, 2-peer ring of 6 agents: the library's ||alpha G(k)||_F of every
    # round against the oracle's (the norm of X - Y, its own RMSProp steps), and the measured distance from
    # consensus under the bound of Proposition 1 built from the LIBRARY's norms, with each round's contraction
    # factor (second singular value of the oracle's dense mixing matrix) and with their maximum as the constant beta
    from paper_1906_04585_b200 import binding as B
    from paper_1906_04585_b200 import learner as LM
    w = GI.WORKLOADS[0].scaled(n_agents=6, topo_kind=R.RING, topo_peers=2)
    net = oracle_net(w)
    L = _learner(w)
    ohp = oracle_hp(L.hp)
    with pytest.raises(B.GalaError):
        B.gala_update_norm(L.ctx)                 # nothing tracked yet
    B.gala_track_updates(L.ctx, True)
    p0 = GI.init_params(GI.net_tensors(w), w.seed)
    for i in range(w.n_agents):
        L.set_state(i, params=p0, sq_avg=np.zeros(L.d, np.float32))
    X = np.tile(p0.astype(np.float64), (w.n_agents, 1))
    V = np.zeros_like(X)
    assert B.gala_consensus_distance(L.ctx) == 0.0
    steps, s2, Ws = [], [], []
    for k in range(5):
        ros = [GI.rollout(w, i, k) for i in range(w.n_agents)]
        L.step_sync([LM.DeviceRollout(r) for r in ros])
        G = np.stack([R.learner_grad(net, X[i], ros[i], ohp)["grad"] for i in range(w.n_agents)])
        Xn, V, Y = R.sweep_sync(X, G, V, ohp, w.topo_kind, w.topo_peers, k)
        want = np.linalg.norm(Y - X)
        got = B.gala_update_norm(L.ctx)
        assert abs(got - want) <= 5 * TOL_FP32_NET * want, (k, got, want)
        steps.append(got)
        s2.append(np.linalg.svd(R.mixing_matrix(w.topo_kind, w.topo_peers, w.n_agents, k), compute_uv=False)[1])
        dist = B.gala_consensus_distance(L.ctx)
        assert abs(dist - R.consensus_distance(Xn)) <= 5 * TOL_FP32_NET * dist + 1e-7
        assert 0.0 < dist <= R.prop1_bound(steps, s2)[k] * (1 + 1e-4)
        assert dist <= R.prop1_bound(steps, max(s2))[k] * (1 + 1e-4)
        # the proof's own form: step s weighted by the norm of (W_k ... W_s - 11^T / n)
        Ws.append(R.mixing_matrix(w.topo_kind, w.topo_peers, w.n_agents, k))
        P, tot = np.eye(w.n_agents), 0.0
        for s_ in range(k, -1, -1):
            P = P @ Ws[s_]
            tot += np.linalg.norm(P - 1.0 / w.n_agents, 2) * steps[s_]
        assert dist <= tot * (1 + 1e-4) and tot <= R.prop1_bound(steps, s2)[k] * (1 + 1e-9)
        X = Xn
    B.gala_track_updates(L.ctx, False)
    with pytest.raises(B.GalaError):
        B.gala_update_norm(L.ctx)
    L.close()


def test_staleness_bound_waits_for_the_in_peer():
    from paper_1906_04585_b200 import binding as B
    from paper_1906_04585_b200 import learner as LM
    w = GI.WORKLOADS[0].scaled(n_agents=2)
    L = _learner(w, staleness_tau=1)
    dev = [LM.DeviceRollout(GI.rollout(w, i, 0)) for i in range(2)]
    # agent 0 alone: two iterations may pass without a message (tau = 1) ...
    for _ in range(2):
        L.learn(0, dev[0]); L.gossip(0)
        assert not B.gala_last_mix(L.ctx, 0)[2]
    # ... the third finds the bound exceeded and nothing published by its in-peer: refused, nothing enqueued
    L.learn(0, dev[0])
    with pytest.raises(B.GalaError) as ei:
        L.gossip(0)
    assert ei.value.status == B.GALA_ETIMEOUT
    assert B.gala_stats(L.ctx, 0)["version"] == 2
    # the in-peer publishes behind a 20 ms straggler delay: agent 0 now WAITS for that snapshot and averages
    B.gala_delay(L.ctx, 1, 20000)
    L.learn(1, dev[1]); L.gossip(1)
    L.gossip(0)
    peers, vers, mixed = B.gala_last_mix(L.ctx, 0)
    assert mixed and peers == [1] and vers == [1]
    st = B.gala_stats(L.ctx, 0)
    assert st["stale_waits"] == 1 and st["mixes"] == 1 and st["version"] == 3
    # with a deadline shorter than the delay the call gives up instead
    B.gala_set_stale_timeout(L.ctx, 2)
    for _ in range(2):
        L.learn(0, dev[0]); L.gossip(0)
    B.gala_delay(L.ctx, 1, 50000)
    L.learn(1, dev[1]); L.gossip(1)
    L.learn(0, dev[0])
    with pytest.raises(B.GalaError) as ei:
        L.gossip(0)
    assert ei.value.status == B.GALA_ETIMEOUT
    L.sync()
    L.gossip(0)                         # the snapshot has landed meanwhile
    assert B.gala_last_mix(L.ctx, 0)[2]
    L.close()


def test_losses_all_agrees_with_per_agent_reads_and_graph_replay_repeats_the_step():
    """Three rounds on the SAME rollout buffers from the same state: the first is launched kernel by kernel, the
    second is captured into a graph, the third replays it.  All three must give the same gradient bit for
    bit, and the batched read of the losses must equal the per-agent reads."""
    from paper_1906_04585_b200 import binding as B, learner as LM
    w = GI.WORKLOADS[1].scaled(n_agents=3, n_envs=2, n_steps=3)
    L = _learner(w)
    p0 = GI.init_params(GI.net_tensors(w), w.seed)
    dev = [LM.DeviceRollout(GI.rollout(w, i, 0)) for i in range(w.n_agents)]
    grads, losses, counted = [], [], []
    for k in range(3):
        for i in range(w.n_agents):
            L.set_state(i, params=p0, sq_avg=np.zeros(L.d, np.float32), rnd=0)
        n0 = B.gala_launch_count(L.ctx)
        L.step_sync(dev)
        L.sync()
        counted.append(B.gala_launch_count(L.ctx) - n0)
        grads.append([L.get_grad(i) for i in range(w.n_agents)])
        la = B.gala_losses_all(L.ctx, w.n_agents)
        for i in range(w.n_agents):
            np.testing.assert_array_equal(la[i], np.array(B.gala_losses(L.ctx, i), np.float32))
        losses.append(la.copy())
    assert counted[0] > 10 and counted[1] == counted[0] and counted[2] == counted[0]   # replayed kernels are counted too
    for k in (1, 2):
        np.testing.assert_array_equal(losses[k], losses[0])
        for i in range(w.n_agents):
            np.testing.assert_array_equal(grads[k][i], grads[0][i])
    # and with the replay switched off
    B.gala_set_graphs(L.ctx, False)
    for i in range(w.n_agents):
        L.set_state(i, params=p0, sq_avg=np.zeros(L.d, np.float32), rnd=0)
    L.step_sync(dev)
    L.sync()
    for i in range(w.n_agents):
        np.testing.assert_array_equal(L.get_grad(i), grads[0][i])
    L.close()


def test_rollout_batch_gives_the_same_round_as_separate_rollouts():
    """All agents' rollouts in one buffer per field (per-agent pointers into it) against one buffer set per agent."""
    from paper_1906_04585_b200 import learner as LM
    w = GI.WORKLOADS[1].scaled(n_agents=3, n_envs=2, n_steps=2)
    p0 = GI.init_params(GI.net_tensors(w), w.seed)
    ros = [GI.rollout(w, i, 0) for i in range(w.n_agents)]
    grads = []
    for batch in (False, True):
        L = _learner(w)
        for i in range(w.n_agents):
            L.set_state(i, params=p0, sq_avg=np.zeros(L.d, np.float32), rnd=0)
        dev = LM.RolloutBatch(ros) if batch else [LM.DeviceRollout(r) for r in ros]
        assert len(dev) == w.n_agents
        L.step_sync(dev)
        L.sync()
        grads.append([L.get_grad(i) for i in range(w.n_agents)])
        L.close()
    for i in range(w.n_agents):
        np.testing.assert_array_equal(grads[0][i], grads[1][i])
