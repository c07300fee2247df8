"""GPU parity at the full sizes of the measured workloads, in the launch configuration the
benchmark times (one synchronous round for all agents), on sampled agents that the oracle can
recompute in seconds; and the asynchronous workload's invariants at full size."""
import numpy as np
import pytest

import gala_inputs as GI
from oracle import reference as R
from tests.helpers import TOL_BF16, assert_close, assert_grad_close, oracle_hp, oracle_net, tie_allowance

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def _run_sync_round(w, sampled):
    from paper_1906_04585_b200 import binding as B
    from paper_1906_04585_b200 import learner as LM
    net = oracle_net(w)
    L = LM.Learner(w.n_agents, w.topo_kind, w.topo_peers, w.net_kind, w.n_actions, w.n_envs, w.n_steps)
    ohp = oracle_hp(L.hp)
    p0 = GI.init_params(GI.net_tensors(w), w.seed)
    for i in range(w.n_agents):
        L.set_state(i, params=p0, sq_avg=np.zeros(L.d, np.float32))
    dev = [LM.DeviceRollout(GI.rollout(w, i, 0)) for i in range(w.n_agents)]
    L.step_sync(dev)
    L.sync()
    S, Bn, A = w.n_envs * w.n_steps, w.n_envs * (w.n_steps + 1), w.n_actions
    if w.n_agents <= 16:
        # the optimiser / gossip stage of the full-size launch on its own: replayed in the oracle from the gradient
        # and norm the library computed, all agents, parameters and second moments to 1e-5, bf16 copy bit for bit
        from tests.test_gpu_learner import replay_sweep_from_library_gradient
        X0 = np.tile(p0.astype(np.float64), (w.n_agents, 1))
        replay_sweep_from_library_gradient(L, B, w, X0, np.zeros_like(X0), ohp, 0)
    # the oracle recomputes the sampled agents and their in-peers of round 0
    need = sorted(set(sampled) | {j for i in sampled for j in R.in_peers(w.topo_kind, w.topo_peers, w.n_agents, 0, i)})
    x0 = p0.astype(np.float64)
    Y = {}
    for i in need:
        ro = GI.rollout(w, i, 0)
        info = R.learner_grad(net, x0, ro, ohp, workers=8)
        assert_close("logits[%d]" % i, L.debug(i, 0, Bn * A), info["logits"], TOL_BF16)
        assert_close("values[%d]" % i, L.debug(i, 1, Bn), info["values"], TOL_BF16)
        assert_close("returns[%d]" % i, L.debug(i, 2, S), info["G"], TOL_BF16)
        # every gradient element within 2e-2 (|g_i| + rms) of the oracle's, except what the gates that the
        # oracle's own two evaluations (exact sums, float32 sums) disagree on can move
        allow = tie_allowance(net, x0, ro["obs"].reshape(Bn, -1)[:S])
        out = assert_grad_close("grad[%d]" % i, L.get_grad(i), info["grad"], net, TOL_BF16, max_outliers=allow)
        print("%s agent %d: %d gradient elements outside the per-element bound, %d allowed" % (w.name, i, out, allow))
        ls = B.gala_losses(L.ctx, i)
        for q in range(3):
            assert abs(ls[q] - info["losses"][q]) <= TOL_BF16 * (abs(info["losses"][q]) + 1.0)
        Y[i] = R.sweep_replay(x0, info["grad"], np.zeros_like(x0), ohp, None)
    for i in sampled:
        peers = R.in_peers(w.topo_kind, w.topo_peers, w.n_agents, 0, i)
        assert L.in_peers(0, i) == peers
        want = R.mix(Y[i][2], [Y[j][2] for j in peers])
        got = L.get_params(i).astype(np.float64)
        assert np.linalg.norm(got - want) <= TOL_BF16 * np.linalg.norm(want)
        du = np.linalg.norm((got - x0) - (want - x0)) / np.linalg.norm(want - x0)
        assert du <= 0.3, du
        v = L.get_sq_avg(i).astype(np.float64)
        assert np.linalg.norm(v - Y[i][1]) <= 2 * TOL_BF16 * np.linalg.norm(Y[i][1])
    # properties that hold at any size: all agents finite, and with identical initialisation the
    # parameters stay within the step-size ball around their mean (Prop. 1 with one step)
    X = np.stack([L.get_params(i) for i in range(w.n_agents)]).astype(np.float64)
    assert np.isfinite(X).all()
    step = np.abs(X - x0).max()
    assert step <= 10.5 * float(L.hp.lr)      # |lr g / (sqrt(0.01 g^2) + eps)| < 10 lr
    L.close()


def test_c2_full_round_all_agents():
    w = GI.WORKLOADS[1]
    _run_sync_round(w, sampled=list(range(w.n_agents)))


def test_c3_full_round_sampled_agents():
    _run_sync_round(GI.WORKLOADS[2], sampled=[4, 11])


def test_c5_full_round_sampled_agents():
    _run_sync_round(GI.WORKLOADS[4], sampled=[37])


def test_c5_async_streams_invariants():
    """64 agents on their own streams, uneven progress and injected straggler delays, nothing
    synchronised between calls: every consumed snapshot must be a completed, published version
    that is newer than the one consumed before, mixes + skips must add up, and all parameters
    must stay finite and close to each other."""
    from paper_1906_04585_b200 import binding as B
    from paper_1906_04585_b200 import learner as LM
    w = GI.WORKLOADS[4]
    n = w.n_agents
    L = LM.Learner(n, w.topo_kind, w.topo_peers, w.net_kind, w.n_actions, w.n_envs, w.n_steps)
    p0 = GI.init_params(GI.net_tensors(w), w.seed)
    for i in range(n):
        L.set_state(i, params=p0, sq_avg=np.zeros(L.d, np.float32))
    dev = [LM.DeviceRollout(GI.rollout(w, i, 0)) for i in range(n)]
    rng = np.random.default_rng(w.seed)
    version = [0] * n
    rnd = [0] * n
    consumed = [[0] * n for _ in range(n)]
    mixes = skipped = 0
    iters = 3
    calls = []
    for _ in range(iters):
        calls += list(rng.permutation(n))
    calls += [0, 0, 5, 5, 5]           # some agents run ahead
    for i in calls:
        i = int(i)
        B.gala_delay(L.ctx, i, int(rng.exponential(300.0)))
        L.learn(i, dev[i])
        L.gossip(i)
        peers, vers, mixed = B.gala_last_mix(L.ctx, i)
        assert peers == R.in_peers(w.topo_kind, w.topo_peers, n, rnd[i], i)
        if mixed:
            mixes += 1
            for pj, vj in zip(peers, vers):
                assert 1 <= vj <= version[pj]            # published ...
                assert vj >= version[pj] - 1             # ... and still held (newest or the one before)
                assert vj > consumed[i][pj]              # fresh
                consumed[i][pj] = vj
        else:
            skipped += 1
            assert all(v == 0 for v in vers)
        version[i] += 1
        rnd[i] += 1
    L.sync()
    stats = [B.gala_stats(L.ctx, i) for i in range(n)]
    assert sum(s["mixes"] for s in stats) == mixes and sum(s["skipped"] for s in stats) == skipped
    assert mixes + skipped == len(calls) and mixes > 0
    assert [s["version"] for s in stats] == version and [s["rounds"] for s in stats] == rnd
    assert sum(s["frames"] for s in stats) == len(calls) * w.n_envs * w.n_steps
    X = np.stack([L.get_params(i) for i in range(n)]).astype(np.float64)
    assert np.isfinite(X).all()
    # identical start, steps bounded by ~10 lr per element and averaging only contracts: every agent
    # stays within (number of its steps) x 10 lr of the start
    for i in range(n):
        assert np.abs(X[i] - p0).max() <= 10.5 * float(L.hp.lr) * max(rnd) + 1e-6
    # a snapshot that is still held can be read back and equals a published version
    snap = np.empty(L.d, np.float32)
    B.gala_get_snapshot(L.ctx, 0, version[0], snap)
    assert np.isfinite(snap).all()
    with pytest.raises(B.GalaError):
        B.gala_get_snapshot(L.ctx, 0, version[0] - 2, snap)
    L.close()
