"""Seeded synthetic inputs for the GALA-A2C learner step.

This module only draws numbers: observations, actions, rewards, episode-end
flags, uniforms for action sampling, initial parameter / optimiser-state /
gradient vectors.  It holds none of the method's arithmetic and is the one
module shared by the CPU oracle's tests and the CUDA path's tests and
benchmark.  Every stream is a Philox counter-based generator keyed by
(BASE_SEED + workload index, stream id), so any piece can be regenerated
independently and identically on any machine.

The workloads stand in for the paper's Atari setting (84x84 grayscale frames,
4 stacked, 16 simulators per learner, horizon 5, rewards clipped to [-1, 1];
Table 2 and Appendix C.2), which needs an emulator that is not available.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Sequence, Tuple

import numpy as np

BASE_SEED = 190604585

RING, EXP, COMPLETE = 0, 1, 2


@dataclass(frozen=True)
class Workload:
    index: int                  # position in the workload list (0-based)
    name: str
    n_agents: int
    topo_kind: int
    topo_peers: int
    net_kind: str               # "mlp" | "conv"
    n_actions: int
    n_envs: int
    n_steps: int
    reward: str                 # "bernoulli" | "ternary"
    done_p: float
    obs_dim: int = 8            # mlp only
    hidden: int = 64            # mlp only
    sweep_only_d: int = 0       # >0: optimiser/gossip microbenchmark, no network

    @property
    def seed(self) -> int:
        return BASE_SEED + self.index

    @property
    def frames_per_round(self) -> int:
        return self.n_agents * self.n_envs * self.n_steps

    def scaled(self, **kw) -> "Workload":
        """Same recipe at other sizes (for tests that must finish in seconds)."""
        d = dict(self.__dict__)
        d.update(kw)
        return Workload(**d)


WORKLOADS: Tuple[Workload, ...] = (
    Workload(0, "c1_mlp_ring_n4", 4, RING, 1, "mlp", 4, 16, 5, "bernoulli", 0.01),
    Workload(1, "c2_conv_exp_n8", 8, EXP, 1, "conv", 6, 16, 5, "bernoulli", 0.01),
    Workload(2, "c3_conv_exp_n16", 16, EXP, 1, "conv", 18, 32, 20, "ternary", 0.005),
    Workload(3, "c4_sweep_n32", 32, EXP, 1, "none", 0, 0, 0, "bernoulli", 0.0, sweep_only_d=1_700_000),
    Workload(4, "c5_conv_async_n64", 64, EXP, 1, "conv", 18, 64, 5, "bernoulli", 0.01),
)


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed & 0xFFFFFFFFFFFFFFFF, stream]))


# stream ids
_S_OBS, _S_ACT, _S_REW, _S_DONE, _S_UNI, _S_PARAM, _S_GRAD, _S_SQ = range(8)


def obs_shape(w: Workload) -> Tuple[int, ...]:
    return (84, 84, 4) if w.net_kind == "conv" else (w.obs_dim,)


def rollout(w: Workload, agent: int, rnd: int = 0) -> Dict[str, np.ndarray]:
    """One agent's rollout for one round: obs [T+1,E,...] (uint8 frames uniform
    in {0..255}, or float32 N(0,1) vectors), actions [T,E] int32 uniform,
    rewards [T,E] float32, dones [T,E] uint8."""
    T, E = w.n_steps, w.n_envs
    sub = (agent << 20) + rnd
    ro = _rng(w.seed, (_S_OBS << 40) + sub)
    if w.net_kind == "conv":
        obs = ro.integers(0, 256, size=(T + 1, E) + obs_shape(w), dtype=np.uint8)
    else:
        obs = ro.standard_normal(size=(T + 1, E) + obs_shape(w), dtype=np.float32)
    actions = _rng(w.seed, (_S_ACT << 40) + sub).integers(0, w.n_actions, size=(T, E), dtype=np.int32)
    rr = _rng(w.seed, (_S_REW << 40) + sub)
    if w.reward == "bernoulli":
        rewards = (rr.random(size=(T, E)) < 0.1).astype(np.float32)
    else:
        u = rr.random(size=(T, E))
        rewards = np.where(u < 0.05, -1.0, np.where(u < 0.95, 0.0, 1.0)).astype(np.float32)
    dones = (_rng(w.seed, (_S_DONE << 40) + sub).random(size=(T, E)) < w.done_p).astype(np.uint8)
    return dict(obs=obs, actions=actions, rewards=rewards, dones=dones)


def uniforms(w: Workload, agent: int, rnd: int, count: int) -> np.ndarray:
    """Pre-drawn uniforms in [0,1) for inverse-CDF action sampling, float32."""
    return _rng(w.seed, (_S_UNI << 40) + (agent << 20) + rnd).random(size=count, dtype=np.float32)


def init_params(tensors: Sequence[Tuple[int, int]], seed: int, agent: int = 0) -> np.ndarray:
    """Flat float32 vector: for each (size, fan_in) in order, `size` draws of
    U(-1,1)/sqrt(fan_in) (fan_in <= 0: zeros, used for biases)."""
    r = _rng(seed, (_S_PARAM << 40) + agent)
    parts = []
    for size, fan_in in tensors:
        if fan_in <= 0:
            parts.append(np.zeros(size, dtype=np.float32))
        else:
            parts.append(((r.random(size=size, dtype=np.float32) * 2.0 - 1.0)
                          / np.float32(np.sqrt(fan_in))).astype(np.float32))
    return np.concatenate(parts) if parts else np.zeros(0, np.float32)


def net_tensors(w: Workload) -> List[Tuple[int, int]]:
    """(size, fan_in) of every tensor of the workload's network in flat order:
    per trunk layer W then b (fan_in 0), then policy W, b, value W, b.
    Small random biases are used (fan_in of the layer) so that bias gradients
    and bias handling are exercised."""
    out: List[Tuple[int, int]] = []
    if w.net_kind == "conv":
        h, c = 84, 4
        for k, s, co in ((8, 4, 32), (4, 2, 64), (3, 1, 64)):
            fan = k * k * c
            out += [(co * fan, fan), (co, fan)]
            h, c = (h - k) // s + 1, co
        feat = h * h * c
        hid = [512]
    else:
        feat = w.obs_dim
        hid = [w.hidden, w.hidden]
    for hdim in hid:
        out += [(hdim * feat, feat), (hdim, feat)]
        feat = hdim
    out += [(w.n_actions * feat, feat), (w.n_actions, feat), (feat, feat), (1, feat)]
    return out


def sweep_state(n_agents: int, d: int, seed: int, rnd: int = 0):
    """Optimiser/gossip microbenchmark inputs, float32 [n,d] each:
    x ~ N(0, std 0.01), g ~ N(0, std 1e-3), v ~ U(0, 1e-4)."""
    x = (_rng(seed, (_S_PARAM << 40) + 1).standard_normal(size=(n_agents, d), dtype=np.float32)
         * np.float32(0.01))
    g = (_rng(seed, (_S_GRAD << 40) + rnd).standard_normal(size=(n_agents, d), dtype=np.float32)
         * np.float32(1e-3))
    v = _rng(seed, (_S_SQ << 40) + 1).random(size=(n_agents, d), dtype=np.float32) * np.float32(1e-4)
    return x, g, v


# ----------------------------------------------------------------------------- synthetic environment
# Counter-based stand-in for the simulators in the closed actor loop: a pure function of
# (seed, agent, environment, step) on the SplitMix64 output function.  No arithmetic of the method
# lives here; the CUDA library has its own statement of the same definition.
_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)


def _sm64(z: np.ndarray) -> np.ndarray:
    z = np.asarray(z, dtype=np.uint64)
    with np.errstate(over="ignore"):
        z = z + np.uint64(0x9E3779B97F4A7C15)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
    return z ^ (z >> np.uint64(31))


def synthetic_env(seed: int, agent: int, n_envs: int, step: int, n_actions: int, frames: bool, obs_dim: int = 8,
                  actions: Optional[np.ndarray] = None) -> Dict[str, np.ndarray]:
    """Observation [E,...] and action-draw uniform [E] of `step`; with `actions` [E] also the reward and the
    done flag of the transition taken at `step`."""
    with np.errstate(over="ignore"):
        env = np.arange(n_envs, dtype=np.uint64)
        base = _sm64(_sm64(_sm64(np.uint64(seed & 0xFFFFFFFFFFFFFFFF) + np.uint64(agent)) + env) + np.uint64(step))
        out = {}
        out["uniforms"] = ((_sm64(base + (np.uint64(3) << np.uint64(56))) >> np.uint64(40)).astype(np.float32)
                           * np.float32(2.0 ** -24))
        if frames:
            n8 = 84 * 84 * 4 // 8
            words = _sm64(base[:, None] + np.arange(n8, dtype=np.uint64)[None, :])
            out["obs"] = words.view(np.uint8).reshape(n_envs, 84, 84, 4)      # little-endian: byte j%8 of word j/8
        else:
            h = _sm64(base[:, None] + np.arange(obs_dim, dtype=np.uint64)[None, :]) >> np.uint64(40)
            out["obs"] = ((h.astype(np.float32) * np.float32(2.0 ** -23) - np.float32(1.0)) * np.float32(1.7320508))
        if actions is not None:
            hr = _sm64(base + (np.uint64(1) << np.uint64(56)))
            hd = _sm64(base + (np.uint64(2) << np.uint64(56))) >> np.uint64(40)
            out["rewards"] = ((hr % np.uint64(n_actions)).astype(np.int64) == np.asarray(actions, np.int64)).astype(np.float32)
            out["dones"] = (hd < np.uint64(167772)).astype(np.uint8)
    return out
