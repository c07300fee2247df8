"""Convenience wrapper around the C ABI: owns a context and the torch device
buffers of the rollouts it is given.  Marshalling only; every step of the
learner path runs inside libgala.so."""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

from . import binding as B


class DeviceRollout:
    """A rollout resident in device memory (torch tensors keep it alive)."""

    def __init__(self, ro: Dict[str, np.ndarray], device="cuda", pinned: bool = False):
        self.host = None
        if pinned:
            self.host = {k: torch.from_numpy(np.ascontiguousarray(v)).pin_memory() for k, v in ro.items()}
            self.t = {k: torch.empty_like(v, device=device) for k, v in self.host.items()}
            self.upload()
        else:
            self.t = {k: torch.from_numpy(np.ascontiguousarray(v)).to(device) for k, v in ro.items()}
        # The copies above run on torch's stream; the library works on streams of its own that do not
        # order themselves against it, so the data must have landed before the rollout is handed over.
        torch.cuda.current_stream().synchronize()
        self.c = B.make_rollout(self.t["obs"], self.t["actions"], self.t["rewards"], self.t["dones"])

    def upload(self, stream: Optional[torch.cuda.Stream] = None):
        """Host -> device copy of the whole rollout from pinned memory."""
        with torch.cuda.stream(stream) if stream is not None else torch.cuda.stream(torch.cuda.current_stream()):
            for k, v in self.host.items():
                self.t[k].copy_(v, non_blocking=True)

    @property
    def nbytes(self) -> int:
        return sum(v.numel() * v.element_size() for v in self.t.values())


class _RolloutView:
    """One agent's part of a RolloutBatch: the same attribute the library calls need (`c`)."""

    def __init__(self, c):
        self.c = c


class RolloutBatch:
    """The rollouts of all agents of one round in ONE pinned host buffer and ONE device buffer per field, so that
    a round's inputs travel host -> device as four copies (one of them carries all the frames) instead of four per
    agent; each agent still gets its own pointers.  Indexing and iteration give per-agent views."""

    def __init__(self, ros: Sequence[Dict[str, np.ndarray]], device="cuda"):
        keys = ("obs", "actions", "rewards", "dones")
        self.host = {k: torch.from_numpy(np.ascontiguousarray(np.stack([r[k] for r in ros]))).pin_memory() for k in keys}
        self.t = {k: torch.empty_like(v, device=device) for k, v in self.host.items()}
        self.upload()
        torch.cuda.current_stream().synchronize()     # the library's streams do not order themselves against torch's
        self.views = [_RolloutView(B.make_rollout(self.t["obs"][i], self.t["actions"][i], self.t["rewards"][i],
                                                  self.t["dones"][i])) for i in range(len(ros))]

    def upload(self, stream: Optional[torch.cuda.Stream] = None):
        with torch.cuda.stream(stream) if stream is not None else torch.cuda.stream(torch.cuda.current_stream()):
            for k, v in self.host.items():
                self.t[k].copy_(v, non_blocking=True)

    def __len__(self):
        return len(self.views)

    def __getitem__(self, i):
        return self.views[i]

    def __iter__(self):
        return iter(self.views)

    @property
    def nbytes(self) -> int:
        return sum(v.numel() * v.element_size() for v in self.t.values())


class Learner:
    def __init__(self, n_agents: int, topo_kind: int, topo_peers: int, net_kind: str, n_actions: int,
                 n_envs: int, n_steps: int, obs_dim: int = 8, hidden: int = 64, **hp_overrides):
        if not torch.cuda.is_available():
            raise RuntimeError("the GALA learner needs a CUDA device (sm_100a); there is no CPU path")
        torch.cuda.init()
        torch.zeros(1, device="cuda")  # make sure the primary context exists before the library uses it
        self.n = n_agents
        self.topo = B.gala_topology(topo_kind, topo_peers)
        conv = net_kind == "conv"
        self.net = B.gala_net_spec(B.GALA_NET_CONV if conv else B.GALA_NET_MLP, obs_dim, hidden, n_actions,
                                   1 if conv else 0)
        self.hp = B.default_hparams(n_envs, n_steps, **hp_overrides)
        self.ctx = B.gala_create(n_agents, self.topo, self.net, self.hp)
        self.d, self.d_pad = B.gala_param_count(self.ctx)
        self.E, self.T, self.A = n_envs, n_steps, n_actions

    def close(self):
        if self.ctx:
            B.gala_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # state ---------------------------------------------------------------
    def get_params(self, agent: int) -> np.ndarray:
        out = np.empty(self.d, np.float32)
        B.gala_get_state(self.ctx, agent, params=out)
        return out

    def get_sq_avg(self, agent: int) -> np.ndarray:
        out = np.empty(self.d, np.float32)
        B.gala_get_state(self.ctx, agent, sq_avg=out)
        return out

    def get_grad(self, agent: int) -> np.ndarray:
        out = np.empty(self.d, np.float32)
        B.gala_get_state(self.ctx, agent, grad=out)
        return out

    def set_state(self, agent: int, params=None, sq_avg=None, rnd: int = 0):
        p = None if params is None else np.ascontiguousarray(params, np.float32)
        v = None if sq_avg is None else np.ascontiguousarray(sq_avg, np.float32)
        B.gala_set_state(self.ctx, agent, p, v, rnd)

    def set_grad(self, agent: int, grad, clip_coef: float = 1.0):
        B.gala_set_grad(self.ctx, agent, np.ascontiguousarray(grad, np.float32), clip_coef)

    # steps ---------------------------------------------------------------
    def step_sync(self, rollouts: Optional[Sequence[DeviceRollout]]):
        B.gala_step_sync(self.ctx, None if rollouts is None else [r.c for r in rollouts])

    def learn(self, agent: int, ro: DeviceRollout):
        B.gala_learn(self.ctx, agent, ro.c)

    def gossip(self, agent: int):
        B.gala_gossip(self.ctx, agent)

    def learn_many(self, agents: Sequence[int], ros: Sequence[DeviceRollout]):
        B.gala_learn_many(self.ctx, agents, [r.c for r in ros])

    def gossip_many(self, agents: Sequence[int]):
        B.gala_gossip_many(self.ctx, agents)

    def act(self, agent: int, obs: torch.Tensor, uniforms: torch.Tensor):
        torch.cuda.current_stream().synchronize()   # obs / uniforms may still be in flight on torch's stream
        actions = torch.empty(self.E, dtype=torch.int32, device=obs.device)
        values = torch.empty(self.E, dtype=torch.float32, device=obs.device)
        B.gala_act(self.ctx, agent, obs, uniforms, actions, values)
        return actions, values

    def sync(self, timeout_ms: int = -1):
        B.gala_sync_all(self.ctx, timeout_ms)

    def in_peers(self, rnd: int, agent: int) -> List[int]:
        return B.gala_in_peers(self.ctx, rnd, agent)

    def debug(self, agent: int, what: int, count: int) -> np.ndarray:
        return B.gala_debug_read(self.ctx, agent, what, count)

    def launches(self) -> int:
        return B.gala_launch_count(self.ctx)
