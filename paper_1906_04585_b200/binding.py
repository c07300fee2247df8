"""ctypes binding of libgala.so: same names as include/gala.h, argument marshalling only.

Every function raises GalaError when the library returns a negative status.
Pointers may be given as torch tensors (their data_ptr is taken; the tensor
must be contiguous), numpy arrays (host memory), ints or None.  There is no
fallback: if the shared library is missing this module raises on first use.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgala.so")

GALA_OK, GALA_EINVAL, GALA_ENOMEM, GALA_ECUDA, GALA_ETIMEOUT, GALA_ESTATE = 0, -1, -2, -3, -4, -5
GALA_NET_MLP, GALA_NET_CONV = 0, 1
GALA_TOPO_RING, GALA_TOPO_EXP, GALA_TOPO_COMPLETE = 0, 1, 2
_STATUS = {0: "GALA_OK", -1: "GALA_EINVAL", -2: "GALA_ENOMEM", -3: "GALA_ECUDA", -4: "GALA_ETIMEOUT",
           -5: "GALA_ESTATE"}


class GalaError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__("%s: %s" % (_STATUS.get(status, status), msg))
        self.status = status


class gala_net_spec(C.Structure):
    _fields_ = [("kind", C.c_int), ("obs_dim", C.c_int), ("hidden", C.c_int), ("n_actions", C.c_int),
                ("gemm_dtype", C.c_int)]


class gala_topology(C.Structure):
    _fields_ = [("kind", C.c_int), ("peers", C.c_int)]


class gala_hparams(C.Structure):
    _fields_ = [("lr", C.c_float), ("rms_alpha", C.c_float), ("rms_eps", C.c_float), ("gamma", C.c_float),
                ("ent_coef", C.c_float), ("vf_coef", C.c_float), ("max_grad_norm", C.c_float),
                ("n_envs", C.c_int), ("n_steps", C.c_int), ("staleness_tau", C.c_int),
                ("seed", C.c_ulonglong), ("identical_init", C.c_int)]


class gala_rollout(C.Structure):
    _fields_ = [("obs", C.c_void_p), ("actions", C.c_void_p), ("rewards", C.c_void_p), ("dones", C.c_void_p)]


class gala_sweep_item(C.Structure):
    _fields_ = [("agent", C.c_int), ("out_slot", C.c_int), ("n_peers", C.c_int), ("peer", C.c_int * 2),
                ("peer_slot", C.c_int * 2), ("has_grad", C.c_int)]


EXPORTS = (
    "gala_create", "gala_destroy", "gala_act", "gala_learn", "gala_gossip", "gala_step_sync",
    "gala_sync_agent", "gala_sync_all", "gala_in_peers", "gala_get_state", "gala_set_state",
    "gala_set_grad", "gala_param_count", "gala_losses", "gala_stats", "gala_last_mix",
    "gala_get_snapshot", "gala_set_stream", "gala_debug_read", "gala_launch_count",
    "gala_last_error", "gala_gemm_bf16", "gala_sweep_sync", "gala_kernel_classes",
    "gala_kernel_class_name", "gala_profile_enable", "gala_profile_read", "gala_get_stream",
    "gala_gemm_bf16_static", "gala_delay", "gala_consensus_distance", "gala_track_updates", "gala_update_norm", "gala_set_stale_timeout",
    "gala_set_agent_ctas", "gala_set_graphs", "gala_losses_all",
    "gala_actor_loop", "gala_actor_loop_all", "gala_actor_read",
    "gala_learn_many", "gala_gossip_many", "gala_poll_agent", "gala_sweep_agents", "gala_set_group_lanes",
    "gala_debug_wait_runs_out",
)

_lib = None


def lib() -> C.CDLL:
    """Load libgala.so (built by paper_1906_04585_b200.build); raises if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                "%s not found: build it with `python -m paper_1906_04585_b200.build` (needs nvcc, sm_100a). "
                "There is no CPU fallback." % LIB_PATH)
        L = C.CDLL(LIB_PATH)
        vp, i, ll, f = C.c_void_p, C.c_int, C.c_longlong, C.c_float
        sig = {
            "gala_create": (i, [i, C.POINTER(gala_topology), C.POINTER(gala_net_spec), C.POINTER(gala_hparams),
                                C.POINTER(vp)]),
            "gala_destroy": (i, [vp]),
            "gala_act": (i, [vp, i, vp, vp, vp, vp]),
            "gala_learn": (i, [vp, i, C.POINTER(gala_rollout)]),
            "gala_gossip": (i, [vp, i]),
            "gala_learn_many": (i, [vp, C.POINTER(i), C.POINTER(gala_rollout), i]),
            "gala_gossip_many": (i, [vp, C.POINTER(i), i]),
            "gala_poll_agent": (i, [vp, i, C.POINTER(i)]),
            "gala_set_group_lanes": (i, [vp, i]),
            "gala_debug_wait_runs_out": (i, [vp, i, i]),
            "gala_sweep_agents": (i, [vp, vp, vp, vp, vp, i, i, ll, C.POINTER(gala_sweep_item), i,
                                      C.POINTER(gala_hparams), vp]),
            "gala_delay": (i, [vp, i, i]),
            "gala_consensus_distance": (i, [vp, C.POINTER(C.c_double)]),
            "gala_track_updates": (i, [vp, i]),
            "gala_update_norm": (i, [vp, C.POINTER(C.c_double)]),
            "gala_set_stale_timeout": (i, [vp, i]),
            "gala_set_agent_ctas": (i, [vp, i]),
            "gala_set_graphs": (i, [vp, i]),
            "gala_actor_loop": (i, [vp, i, i, C.c_ulonglong]),
            "gala_actor_loop_all": (i, [vp, i, C.c_ulonglong]),
            "gala_actor_read": (i, [vp, i, vp, vp, vp, vp, C.POINTER(C.c_longlong)]),
            "gala_step_sync": (i, [vp, C.POINTER(gala_rollout)]),
            "gala_sync_agent": (i, [vp, i, i]),
            "gala_sync_all": (i, [vp, i]),
            "gala_in_peers": (i, [vp, ll, i, C.POINTER(i), C.POINTER(i)]),
            "gala_get_state": (i, [vp, i, vp, vp, vp, C.POINTER(ll)]),
            "gala_set_state": (i, [vp, i, vp, vp, ll]),
            "gala_set_grad": (i, [vp, i, vp, f]),
            "gala_param_count": (i, [vp, C.POINTER(ll), C.POINTER(ll)]),
            "gala_losses": (i, [vp, i, C.POINTER(f)]),
            "gala_losses_all": (i, [vp, C.POINTER(f)]),
            "gala_stats": (i, [vp, i, C.POINTER(ll)]),
            "gala_last_mix": (i, [vp, i, C.POINTER(i), C.POINTER(ll), C.POINTER(i), C.POINTER(i)]),
            "gala_get_snapshot": (i, [vp, i, ll, vp]),
            "gala_set_stream": (i, [vp, i, vp]),
            "gala_debug_read": (i, [vp, i, i, vp, ll]),
            "gala_launch_count": (ll, [vp]),
            "gala_last_error": (C.c_char_p, [vp]),
            "gala_kernel_classes": (i, []),
            "gala_kernel_class_name": (C.c_char_p, [i]),
            "gala_profile_enable": (i, [vp, C.c_ulonglong]),
            "gala_profile_read": (i, [vp, C.POINTER(C.c_double), C.POINTER(ll), C.POINTER(ll), i]),
            "gala_get_stream": (vp, [vp, i]),
            "gala_gemm_bf16": (i, [vp, vp, vp, i, i, i, i, i, i, i, vp]),
            "gala_gemm_bf16_static": (i, [vp, vp, vp, i, i, i, i, i, i, i, vp, C.c_char_p, i]),
            "gala_sweep_sync": (i, [vp, vp, vp, vp, i, ll, C.POINTER(gala_topology), ll, C.POINTER(gala_hparams), vp]),
        }
        for name, (res, args) in sig.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if isinstance(t, np.ndarray):
        assert t.flags["C_CONTIGUOUS"]
        return t.ctypes.data
    if hasattr(t, "data_ptr"):
        assert t.is_contiguous()
        return t.data_ptr()
    raise TypeError(type(t))


def _check(ctx, rc: int):
    if rc < 0:
        msg = lib().gala_last_error(ctx).decode() if ctx else ""
        raise GalaError(rc, msg)
    return rc


def make_rollout(obs, actions, rewards, dones) -> gala_rollout:
    return gala_rollout(_ptr(obs), _ptr(actions), _ptr(rewards), _ptr(dones))


def gala_create(n_agents: int, topo: gala_topology, net: gala_net_spec, hp: gala_hparams) -> C.c_void_p:
    h = C.c_void_p()
    rc = lib().gala_create(n_agents, C.byref(topo), C.byref(net), C.byref(hp), C.byref(h))
    if rc < 0:
        msg = lib().gala_last_error(h).decode() if h else "invalid argument"
        if h:
            lib().gala_destroy(h)
        raise GalaError(rc, msg)
    return h


def gala_destroy(ctx):
    _check(None, lib().gala_destroy(ctx))


def gala_act(ctx, agent: int, obs, uniforms, actions, values):
    _check(ctx, lib().gala_act(ctx, agent, _ptr(obs), _ptr(uniforms), _ptr(actions), _ptr(values)))


def gala_learn(ctx, agent: int, rollout: gala_rollout):
    _check(ctx, lib().gala_learn(ctx, agent, C.byref(rollout)))


def gala_gossip(ctx, agent: int):
    _check(ctx, lib().gala_gossip(ctx, agent))


def gala_learn_many(ctx, agents: Sequence[int], rollouts: Sequence[gala_rollout]):
    m = len(agents)
    assert len(rollouts) == m
    ids = (C.c_int * m)(*agents)
    arr = rollouts if isinstance(rollouts, C.Array) else (gala_rollout * m)(*rollouts)
    _check(ctx, lib().gala_learn_many(ctx, ids, arr, m))


def gala_gossip_many(ctx, agents: Sequence[int]):
    m = len(agents)
    _check(ctx, lib().gala_gossip_many(ctx, (C.c_int * m)(*agents), m))


def gala_poll_agent(ctx, agent: int) -> bool:
    """True while work enqueued for the agent is still running."""
    busy = C.c_int()
    _check(ctx, lib().gala_poll_agent(ctx, agent, C.byref(busy)))
    return bool(busy.value)


def gala_set_group_lanes(ctx, lanes: int):
    _check(ctx, lib().gala_set_group_lanes(ctx, lanes))


def gala_debug_wait_runs_out(ctx, agent: int, polls: int):
    _check(ctx, lib().gala_debug_wait_runs_out(ctx, agent, polls))


def gala_delay(ctx, agent: int, usec: int):
    _check(ctx, lib().gala_delay(ctx, agent, usec))


def gala_consensus_distance(ctx) -> float:
    out = C.c_double()
    _check(ctx, lib().gala_consensus_distance(ctx, C.byref(out)))
    return out.value


def gala_track_updates(ctx, on: bool):
    _check(ctx, lib().gala_track_updates(ctx, 1 if on else 0))


def gala_update_norm(ctx) -> float:
    out = C.c_double()
    _check(ctx, lib().gala_update_norm(ctx, C.byref(out)))
    return out.value


def gala_actor_loop(ctx, agent: int, iterations: int, env_seed: int):
    _check(ctx, lib().gala_actor_loop(ctx, agent, iterations, env_seed))


def gala_actor_loop_all(ctx, iterations: int, env_seed: int):
    _check(ctx, lib().gala_actor_loop_all(ctx, iterations, env_seed))


def gala_actor_read(ctx, agent: int, n_envs: int, n_steps: int, obs_shape, obs_dtype):
    """Host copies of the agent's last closed-loop rollout: dict(obs, actions, rewards, dones), next step."""
    obs = np.empty((n_steps + 1, n_envs) + tuple(obs_shape), dtype=obs_dtype)
    actions = np.empty((n_steps, n_envs), dtype=np.int32)
    rewards = np.empty((n_steps, n_envs), dtype=np.float32)
    dones = np.empty((n_steps, n_envs), dtype=np.uint8)
    nxt = C.c_longlong()
    _check(ctx, lib().gala_actor_read(ctx, agent, obs.ctypes.data, actions.ctypes.data, rewards.ctypes.data,
                                      dones.ctypes.data, C.byref(nxt)))
    return dict(obs=obs, actions=actions, rewards=rewards, dones=dones), int(nxt.value)


def gala_set_graphs(ctx, mode):
    """0 / False: never; 1 / True: graph replay in the synchronous round; 2: also in the per-agent calls."""
    _check(ctx, lib().gala_set_graphs(ctx, int(mode)))


def gala_set_agent_ctas(ctx, ctas: int):
    _check(ctx, lib().gala_set_agent_ctas(ctx, ctas))


def gala_set_stale_timeout(ctx, timeout_ms: int):
    _check(ctx, lib().gala_set_stale_timeout(ctx, timeout_ms))


def gala_step_sync(ctx, rollouts: Optional[Sequence[gala_rollout]]):
    if rollouts is None:
        _check(ctx, lib().gala_step_sync(ctx, None))
        return
    arr = rollouts if isinstance(rollouts, C.Array) else (gala_rollout * len(rollouts))(*rollouts)
    _check(ctx, lib().gala_step_sync(ctx, arr))


def gala_sync_agent(ctx, agent: int, timeout_ms: int = -1):
    _check(ctx, lib().gala_sync_agent(ctx, agent, timeout_ms))


def gala_sync_all(ctx, timeout_ms: int = -1):
    _check(ctx, lib().gala_sync_all(ctx, timeout_ms))


def gala_in_peers(ctx, rnd: int, agent: int):
    peers = (C.c_int * 4)()
    n = C.c_int()
    _check(ctx, lib().gala_in_peers(ctx, rnd, agent, peers, C.byref(n)))
    return [peers[j] for j in range(n.value)]


def gala_param_count(ctx):
    d, dp = C.c_longlong(), C.c_longlong()
    _check(ctx, lib().gala_param_count(ctx, C.byref(d), C.byref(dp)))
    return d.value, dp.value


def gala_get_state(ctx, agent: int, params=None, sq_avg=None, grad=None) -> int:
    rnd = C.c_longlong()
    _check(ctx, lib().gala_get_state(ctx, agent, _ptr(params), _ptr(sq_avg), _ptr(grad), C.byref(rnd)))
    return rnd.value


def gala_set_state(ctx, agent: int, params=None, sq_avg=None, rnd: int = 0):
    _check(ctx, lib().gala_set_state(ctx, agent, _ptr(params), _ptr(sq_avg), rnd))


def gala_set_grad(ctx, agent: int, grad, clip_coef: float = 1.0):
    _check(ctx, lib().gala_set_grad(ctx, agent, _ptr(grad), clip_coef))


def gala_losses(ctx, agent: int):
    out = (C.c_float * 4)()
    _check(ctx, lib().gala_losses(ctx, agent, out))
    return [out[j] for j in range(4)]


def gala_losses_all(ctx, n_agents: int) -> np.ndarray:
    out = np.empty((n_agents, 4), dtype=np.float32)
    _check(ctx, lib().gala_losses_all(ctx, out.ctypes.data_as(C.POINTER(C.c_float))))
    return out


def gala_stats(ctx, agent: int):
    out = (C.c_longlong * 8)()
    _check(ctx, lib().gala_stats(ctx, agent, out))
    return dict(frames=out[0], rounds=out[1], mixes=out[2], skipped=out[3], staleness_sum=out[4],
                staleness_max=out[5], version=out[6], stale_waits=out[7])


def gala_last_mix(ctx, agent: int):
    peers, vers = (C.c_int * 4)(), (C.c_longlong * 4)()
    n, mixed = C.c_int(), C.c_int()
    _check(ctx, lib().gala_last_mix(ctx, agent, peers, vers, C.byref(n), C.byref(mixed)))
    return [peers[j] for j in range(n.value)], [vers[j] for j in range(n.value)], bool(mixed.value)


def gala_get_snapshot(ctx, agent: int, version: int, out):
    _check(ctx, lib().gala_get_snapshot(ctx, agent, version, _ptr(out)))


def gala_set_stream(ctx, agent: int, cuda_stream: Optional[int]):
    _check(ctx, lib().gala_set_stream(ctx, agent, cuda_stream))


def gala_debug_read(ctx, agent: int, what: int, count: int) -> np.ndarray:
    out = np.empty(count, dtype=np.float32)
    _check(ctx, lib().gala_debug_read(ctx, agent, what, out.ctypes.data, count))
    return out


def gala_launch_count(ctx) -> int:
    return int(lib().gala_launch_count(ctx))


def gala_kernel_classes() -> int:
    return int(lib().gala_kernel_classes())


def gala_kernel_class_name(k: int) -> str:
    return lib().gala_kernel_class_name(k).decode()


def gala_profile_enable(ctx, mask: int):
    _check(ctx, lib().gala_profile_enable(ctx, mask))


def gala_profile_read(ctx, reset: bool = True):
    """{class name: (summed ms of timed launches, timed launches, launches issued)}"""
    n = gala_kernel_classes()
    ms, timed, launches = (C.c_double * n)(), (C.c_longlong * n)(), (C.c_longlong * n)()
    _check(ctx, lib().gala_profile_read(ctx, ms, timed, launches, 1 if reset else 0))
    return {gala_kernel_class_name(k): (ms[k], timed[k], launches[k]) for k in range(n)}


def gala_get_stream(ctx, agent: int = -1) -> int:
    return int(lib().gala_get_stream(ctx, agent) or 0)


def gala_last_error(ctx) -> str:
    return lib().gala_last_error(ctx).decode()


def gala_gemm_bf16(A, B, D, groups, M, N, K, a_mn=0, b_mn=0, split_k=1, stream=None):
    rc = lib().gala_gemm_bf16(_ptr(A), _ptr(B), _ptr(D), groups, M, N, K, a_mn, b_mn, split_k, stream)
    if rc < 0:
        raise GalaError(rc, "gala_gemm_bf16")


def gala_gemm_bf16_static(A, B, D, groups, M, N, K, a_mn=0, b_mn=0, split_k=1, stream=None):
    """gala_gemm_bf16 for hosts that cannot allocate device memory: scratch comes from an 8 MiB
    array inside the library (groups*split_k*M*N <= 2 Mi floats when split_k > 1)."""
    buf = C.create_string_buffer(512)
    rc = lib().gala_gemm_bf16_static(_ptr(A), _ptr(B), _ptr(D), groups, M, N, K, a_mn, b_mn, split_k, stream,
                                     buf, len(buf))
    if rc < 0:
        raise GalaError(rc, buf.value.decode())


def gala_sweep_sync(x, g, v, clip, n_agents, d_padded, topo: gala_topology, rnd: int, hp: gala_hparams,
                    stream=None):
    rc = lib().gala_sweep_sync(_ptr(x), _ptr(g), _ptr(v), _ptr(clip), n_agents, d_padded, C.byref(topo), rnd,
                               C.byref(hp), stream)
    if rc < 0:
        raise GalaError(rc, "gala_sweep_sync")


def gala_sweep_agents(x, g, v, snap, clip, n_agents: int, n_slots: int, d_padded: int, items, hp: gala_hparams,
                      stream=None):
    """items: sequence of (agent, out_slot, [(peer, peer_slot), ...], has_grad)."""
    arr = (gala_sweep_item * len(items))()
    for k, (agent, out_slot, peers, has_grad) in enumerate(items):
        arr[k].agent, arr[k].out_slot, arr[k].n_peers, arr[k].has_grad = agent, out_slot, len(peers), int(has_grad)
        for j, (pj, sj) in enumerate(peers):
            arr[k].peer[j], arr[k].peer_slot[j] = pj, sj
    rc = lib().gala_sweep_agents(_ptr(x), _ptr(g), _ptr(v), _ptr(snap), _ptr(clip), n_agents, n_slots, d_padded, arr,
                                 len(items), C.byref(hp), stream)
    if rc < 0:
        raise GalaError(rc, "gala_sweep_agents")


def default_hparams(n_envs: int, n_steps: int, **kw) -> gala_hparams:
    """Table 2 values, with the RMSProp alpha/epsilon of the measured workloads."""
    d = dict(lr=7e-4, rms_alpha=0.99, rms_eps=1e-5, gamma=0.99, ent_coef=0.01, vf_coef=0.5, max_grad_norm=0.5,
             n_envs=n_envs, n_steps=n_steps, staleness_tau=-1, seed=1, identical_init=1)
    d.update(kw)
    return gala_hparams(**d)
