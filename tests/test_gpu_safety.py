"""Two safety nets of the asynchronous mode, neither of which faults or hangs anything.

1. Snapshot contents under real concurrency (Appendix A: one receive slot per in-peer, the newest message
   overwrites): every agent's parameters are a constant vector, no gradient is ever pending, so every published
   snapshot is a constant vector too and every average of constant vectors is one.  Gossip steps are issued
   without any host wait, on the agents' own streams with injected delays, or as grouped calls on two streams.  A
   snapshot slot that is overwritten while a reader is still on it would leave the reader with a vector that is
   NOT constant along the parameter index; and the constant every agent ends with must be the one that the logged
   (in-peer, version) pairs imply, replayed in float32 with the kernel's order of operations: bit for bit.
2. The report of a bounded device-side wait that runs out (Sec. 3's bounded staleness has its host-side
   counterpart tested elsewhere): a wait on a barrier that nothing arrives at gives up after a few polls, the
   error word reaches the host as GALA_ECUDA at the next wait, and the context goes on working.
"""
import numpy as np
import pytest

import gala_inputs as GI
from oracle import reference as R

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def _mods():
    from paper_1906_04585_b200 import binding, learner
    return binding, learner


def _constant_agents(n, peers, lanes=None):
    B, LM = _mods()
    w = GI.WORKLOADS[1].scaled(n_agents=n, n_envs=1, n_steps=1, topo_peers=peers)
    L = LM.Learner(n, w.topo_kind, peers, w.net_kind, w.n_actions, 1, 1)
    if lanes:
        B.gala_set_group_lanes(L.ctx, lanes)
    for i in range(n):
        L.set_state(i, params=np.full(L.d, 1.0 + i, np.float32), sq_avg=np.zeros(L.d, np.float32), rnd=0)
    return B, L, w


def _replay(value, snaps, i, peers, vers, mixed, version):
    """One gossip step without a pending gradient, in float32 with the kernels' order: publish y = x, then
    x = ((y + m0) + m1) * (1 / (1 + p)) if it averaged."""
    y = value[i]
    version[i] += 1
    snaps[(i, version[i])] = y
    if mixed:
        acc = y
        for pj, vj in zip(peers, vers):
            assert 1 <= vj <= version[pj] and (pj, vj) in snaps
            acc = np.float32(acc + snaps[(pj, vj)])
        value[i] = np.float32(acc * np.float32(1.0 / (1.0 + len(peers))))


def _check_constant(L, n, value):
    for i in range(n):
        x = L.get_params(i)
        assert x.min() == x.max(), "agent %d: parameters are not one constant (a snapshot was read while it changed)" % i
        assert x[0] == value[i], (i, x[0], value[i])


@pytest.mark.parametrize("peers", [1, 2])
def test_snapshots_are_never_read_while_they_change_per_agent_streams(peers):
    n = 8
    B, L, w = _constant_agents(n, peers)
    rng = np.random.default_rng(5)
    value = [np.float32(1.0 + i) for i in range(n)]
    snaps, version, rnd = {}, [0] * n, [0] * n
    mixes = 0
    calls = [int(i) for _ in range(40) for i in rng.permutation(n)] + [3] * 6 + [0, 3, 0, 3]
    for i in calls:
        if rng.random() < 0.5:
            B.gala_delay(L.ctx, i, int(rng.integers(1, 60)))
        L.gossip(i)                                   # no host wait anywhere
        p, v, mixed = B.gala_last_mix(L.ctx, i)
        assert p == R.in_peers(w.topo_kind, peers, n, rnd[i], i)
        _replay(value, snaps, i, p, v, mixed, version)
        mixes += int(mixed)
        rnd[i] += 1
    L.sync()
    assert 0 < mixes < len(calls)                     # both outcomes occurred
    _check_constant(L, n, value)
    L.close()


@pytest.mark.parametrize("lanes", [1, 2])
def test_snapshots_are_never_read_while_they_change_grouped_calls(lanes):
    n = 8
    B, L, w = _constant_agents(n, 1, lanes=lanes)
    rng = np.random.default_rng(6 + lanes)
    value = [np.float32(1.0 + i) for i in range(n)]
    snaps, version, rnd = {}, [0] * n, [0] * n
    mixes = total = 0
    for step in range(60):
        if step % 7 == 3:                             # per-agent calls in between: all forms share the slots
            lst = [int(rng.integers(0, n))]
            L.gossip(lst[0])
        else:
            lst = [int(i) for i in rng.permutation(n)[: int(rng.integers(1, n + 1))]]
            L.gossip_many(lst)
        logs = [(i,) + tuple(B.gala_last_mix(L.ctx, i)) for i in lst]
        # every agent of a call decided before anything of the call was published: replay the reads first
        staged = {}
        for i, p, v, mixed in logs:
            assert p == R.in_peers(w.topo_kind, 1, n, rnd[i], i)
            for pj, vj in zip(p, v):
                if mixed:
                    assert vj <= version[pj]          # never a snapshot of the same call
            staged[i] = (p, v, mixed)
        new_value = {}
        for i, (p, v, mixed) in staged.items():
            val = list(value)
            ver = list(version)
            _replay(val, snaps, i, p, v, mixed, ver)
            new_value[i] = (val[i], ver[i])
            mixes += int(mixed)
            total += 1
        for i, (val, ver) in new_value.items():
            value[i], version[i] = val, ver
            rnd[i] += 1
    L.sync()
    assert 0 < mixes <= total
    _check_constant(L, n, value)
    L.close()


def test_a_device_side_wait_that_runs_out_is_reported_and_the_context_goes_on():
    B, LM = _mods()
    w = GI.WORKLOADS[0]
    L = LM.Learner(w.n_agents, w.topo_kind, w.topo_peers, w.net_kind, w.n_actions, w.n_envs, w.n_steps,
                   obs_dim=w.obs_dim, hidden=w.hidden)
    L.sync()                                          # clean to begin with
    B.gala_debug_wait_runs_out(L.ctx, 1, 1000)        # a barrier nobody arrives at: gives up after 1000 polls
    with pytest.raises(B.GalaError) as ei:
        L.sync()
    assert ei.value.status == B.GALA_ECUDA and "wait ran out" in str(ei.value)
    L.sync()                                          # reported once, then cleared
    # the context still works: a synchronous round against the oracle
    net = R.Net.mlp(w.obs_dim, w.hidden, w.n_actions)
    p0 = GI.init_params(GI.net_tensors(w), w.seed)
    for i in range(w.n_agents):
        L.set_state(i, params=p0, sq_avg=np.zeros(L.d, np.float32), rnd=0)
    ros = [GI.rollout(w, i, 0) for i in range(w.n_agents)]
    L.step_sync([LM.DeviceRollout(r) for r in ros])
    L.sync()
    hp = R.HParams(lr=float(L.hp.lr), rms_alpha=float(L.hp.rms_alpha), rms_eps=float(L.hp.rms_eps),
                   gamma=float(L.hp.gamma), ent_coef=float(L.hp.ent_coef), vf_coef=float(L.hp.vf_coef),
                   max_grad_norm=float(L.hp.max_grad_norm))
    X = np.tile(p0.astype(np.float64), (w.n_agents, 1))
    Xn, _, _ = R.sync_round(net, X, np.zeros_like(X), ros, hp, w.topo_kind, w.topo_peers, 0)
    for i in range(w.n_agents):
        assert np.abs(L.get_params(i) - Xn[i]).max() <= 1e-5 * (np.abs(Xn[i]).max() + 1)
    with pytest.raises(B.GalaError):
        B.gala_debug_wait_runs_out(L.ctx, 0, 0)       # poll counts outside 1..100000 are refused
    L.close()
