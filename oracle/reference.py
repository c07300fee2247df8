"""fp64 CPU oracle for the GALA-A2C learner step (arXiv 1906.04585).

TEST INFRASTRUCTURE.  Only the test suite, the smoke check and the
CPU-baseline leg of the benchmark may import this module; the product path
never does, and this module imports nothing from the CUDA package.

The arithmetic lives in ``gala_oracle.c`` (plain C loops, double precision);
this file marshals numpy arrays into it and composes the steps of
Algorithm 1 in the paper's order:

  act / forward           -> ``forward``
  returns and advantages  -> ``returns``           (Sec. 2; Algorithm 1)
  A2C objective, gradient -> ``a2c_loss``, ``backward``   (Eqs. 1-4)
  clip + RMSProp          -> ``clip_coef``, ``rmsprop``   (Table 2)
  broadcast + average     -> ``in_peers``, ``mix``, ``sweep_sync``,
                             ``sweep_replay``  (Algorithm 1 gossip steps and
                             its footnote; Eqs. 5-7 of the appendix)

  distance from consensus -> ``consensus_distance``, ``prop1_bound``
                             (Propositions 1-2)

Topology schedules are integer-only Python.

Parity status: every function here is pinned by tests/test_oracle_*.py to
closed forms, finite differences, brute force or spectral facts, EXCEPT the
asynchronous schedule itself (which peer version a learner happens to see),
which the paper fixes only through invariants: "parity unpinned" for that
choice; ``sweep_replay`` replays a recorded schedule instead.
"""
from __future__ import annotations

import ctypes as C
import math
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

from . import build as _build

_MAXC, _MAXH = 4, 4


class _CNet(C.Structure):
    _fields_ = [
        ("n_conv", C.c_int),
        ("in_h", C.c_int), ("in_w", C.c_int), ("in_c", C.c_int),
        ("ck", C.c_int * _MAXC), ("cs", C.c_int * _MAXC), ("cc", C.c_int * _MAXC),
        ("n_hidden", C.c_int),
        ("hidden", C.c_int * _MAXH),
        ("act", C.c_int),
        ("n_actions", C.c_int),
        ("in_scale", C.c_double),
        ("round_bf16", C.c_int),
        ("sum_f32", C.c_int),
    ]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        dp = C.POINTER(C.c_double)
        L.orc_param_count.restype = C.c_long
        L.orc_param_count.argtypes = [C.POINTER(_CNet)]
        L.orc_param_offsets.restype = C.c_int
        L.orc_param_offsets.argtypes = [C.POINTER(_CNet), C.POINTER(C.c_long)]
        L.orc_forward.restype = C.c_int
        L.orc_forward.argtypes = [C.POINTER(_CNet), dp, dp, C.c_int, dp, dp, C.c_int, dp]
        L.orc_backward.restype = C.c_int
        L.orc_backward.argtypes = [C.POINTER(_CNet), dp, dp, C.c_int, dp, dp, dp]
        L.orc_returns.restype = None
        L.orc_returns.argtypes = [C.c_int, C.c_int, C.c_double, dp, C.POINTER(C.c_ubyte), dp, dp]
        L.orc_a2c_loss.restype = None
        L.orc_a2c_loss.argtypes = [C.c_int, C.c_int, dp, C.POINTER(C.c_int), dp, dp, dp,
                                   C.c_double, C.c_double, dp, dp, dp]
        L.orc_clip_coef.restype = C.c_double
        L.orc_clip_coef.argtypes = [C.c_long, dp, C.c_double, dp]
        L.orc_rmsprop.restype = None
        L.orc_rmsprop.argtypes = [C.c_long, dp, dp, dp, C.c_double, C.c_double, C.c_double,
                                  C.c_double, dp]
        L.orc_mix.restype = None
        L.orc_mix.argtypes = [C.c_long, dp, C.c_int, C.POINTER(dp), dp]
        L.orc_round_bf16.restype = C.c_double
        L.orc_round_bf16.argtypes = [C.c_double]
        L.orc_sample.restype = C.c_int
        L.orc_sample.argtypes = [C.c_int, dp, C.c_double]
        _lib = L
    return _lib


def _dp(a: np.ndarray):
    return a.ctypes.data_as(C.POINTER(C.c_double))


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float64)


# --------------------------------------------------------------------------
# network description
# --------------------------------------------------------------------------
@dataclass
class Net:
    """Trunk of VALID convolutions (NHWC, weights [cout][kh][kw][cin]) and dense
    layers, each followed by `act`; linear policy and value heads on top."""
    in_h: int = 1
    in_w: int = 1
    in_c: int = 8
    convs: Sequence[Tuple[int, int, int]] = ()      # (kernel, stride, cout)
    hidden: Sequence[int] = (64, 64)
    act: str = "tanh"                                # "relu" | "tanh"
    n_actions: int = 4
    in_scale: float = 1.0
    # "bf16 GEMMs, fp32 params": operands of every trunk contraction (weights, stored activations,
    # stored pre-activation gradients) are rounded to bfloat16, sums stay exact.  Chosen so that
    # the ReLU gate, a yes/no decision taken on a stored activation, is taken on the same number
    # by the oracle and by a kernel that stores activations in bf16.  False: exact arithmetic.
    bf16_operands: bool = False
    # Not the method: the same rounded network with every trunk sum formed in float32, term after term, instead of
    # exactly - a second valid evaluation, for measuring how far two implementations that differ only in summation
    # precision drift apart (see gate_flips).
    sum_f32: bool = False

    def with_bf16(self, on: bool = True) -> "Net":
        return replace(self, bf16_operands=on)

    def with_f32_sums(self, on: bool = True) -> "Net":
        return replace(self, sum_f32=on)

    @staticmethod
    def mlp(obs_dim: int = 8, hidden: int = 64, n_actions: int = 4) -> "Net":
        return Net(1, 1, obs_dim, (), (hidden, hidden), "tanh", n_actions, 1.0)

    @staticmethod
    def atari(n_actions: int = 6) -> "Net":
        """Appendix C.2 network at the sizes of the measured workloads."""
        return Net(84, 84, 4, ((8, 4, 32), (4, 2, 64), (3, 1, 64)), (512,), "relu",
                   n_actions, 1.0 / 255.0)

    def c(self) -> _CNet:
        n = _CNet()
        n.n_conv = len(self.convs)
        n.in_h, n.in_w, n.in_c = self.in_h, self.in_w, self.in_c
        for i, (k, s, cc) in enumerate(self.convs):
            n.ck[i], n.cs[i], n.cc[i] = k, s, cc
        n.n_hidden = len(self.hidden)
        for i, h in enumerate(self.hidden):
            n.hidden[i] = h
        n.act = 0 if self.act == "relu" else 1
        n.n_actions = self.n_actions
        n.in_scale = self.in_scale
        n.round_bf16 = 1 if self.bf16_operands else 0
        n.sum_f32 = 1 if self.sum_f32 else 0
        return n

    @property
    def in_size(self) -> int:
        return self.in_h * self.in_w * self.in_c

    def layer_out_shape(self, li: int) -> Tuple[int, ...]:
        h, w, c = self.in_h, self.in_w, self.in_c
        for i, (k, s, cc) in enumerate(self.convs):
            h, w, c = (h - k) // s + 1, (w - k) // s + 1, cc
            if i == li:
                return (h, w, c)
        return (self.hidden[li - len(self.convs)],)


def param_count(net: Net) -> int:
    cn = net.c()
    return int(lib().orc_param_count(C.byref(cn)))


def param_offsets(net: Net) -> Dict[str, int]:
    """Offsets of every tensor in the flat vector, keyed 'L0.W', 'L0.b', ...,
    'pi.W', 'pi.b', 'v.W', 'v.b', plus 'd'."""
    cn = net.c()
    out = (C.c_long * 32)()
    nl = lib().orc_param_offsets(C.byref(cn), out)
    res = {}
    for i in range(nl):
        res["L%d.W" % i], res["L%d.b" % i] = out[2 * i], out[2 * i + 1]
    res["pi.W"], res["pi.b"], res["v.W"], res["v.b"] = (out[2 * nl + j] for j in range(4))
    res["d"] = param_count(net)
    return res


def round_bf16(a) -> np.ndarray:
    """Element-wise round to bfloat16 (nearest even), returned as float64."""
    a = _f64(a)
    out = np.empty_like(a)
    L = lib()
    flat_in, flat_out = a.ravel(), out.ravel()
    for i in range(flat_in.size):
        flat_out[i] = L.orc_round_bf16(float(flat_in[i]))
    return out


def effective_params(net: Net, params) -> np.ndarray:
    """Parameters as the contractions see them: with bf16 operands, the trunk weight tensors are
    rounded to bfloat16 (biases and the two linear heads stay as given)."""
    p = _f64(params).copy()
    if not net.bf16_operands:
        return p
    off = param_offsets(net)
    nl = len(net.convs) + len(net.hidden)
    for i in range(nl):
        lo, hi = off["L%d.W" % i], off["L%d.b" % i]
        f = p[lo:hi].astype(np.float32)
        u = f.view(np.uint32).astype(np.uint64)
        u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
        p[lo:hi] = u.astype(np.uint32).view(np.float32).astype(np.float64)
    return p


# --------------------------------------------------------------------------
# network forward / backward
# --------------------------------------------------------------------------
def forward(net: Net, params, obs, which_layer: Optional[int] = None):
    """obs: [B, ...] raw observations (any numeric dtype).  Returns
    (logits [B,A], values [B]) and, if which_layer is given, also that trunk
    layer's post-activation output [B, ...]."""
    p = effective_params(net, params)
    o = _f64(obs).reshape(len(obs), -1)
    assert o.shape[1] == net.in_size and p.size == param_count(net)
    B = o.shape[0]
    logits = np.empty((B, net.n_actions))
    values = np.empty(B)
    cn = net.c()
    lo = None
    if which_layer is not None:
        lo = np.empty((B,) + net.layer_out_shape(which_layer))
    rc = lib().orc_forward(C.byref(cn), _dp(p), _dp(o), B, _dp(logits), _dp(values),
                           -1 if which_layer is None else which_layer,
                           _dp(lo) if lo is not None else None)
    assert rc == 0
    return (logits, values) if lo is None else (logits, values, lo)


def backward(net: Net, params, obs, dlogits, dvalues) -> np.ndarray:
    p = effective_params(net, params)
    o = _f64(obs).reshape(len(obs), -1)
    dz, dv = _f64(dlogits), _f64(dvalues)
    B = o.shape[0]
    assert dz.shape == (B, net.n_actions) and dv.shape == (B,)
    g = np.zeros(p.size)
    cn = net.c()
    rc = lib().orc_backward(C.byref(cn), _dp(p), _dp(o), B, _dp(dz), _dp(dv), _dp(g))
    assert rc == 0
    return g


# --------------------------------------------------------------------------
# returns, loss
# --------------------------------------------------------------------------
def returns(rewards, dones, v_boot, gamma: float) -> np.ndarray:
    r = _f64(rewards)
    T, E = r.shape
    dn = np.ascontiguousarray(dones, dtype=np.uint8)
    vb = _f64(v_boot)
    G = np.empty((T, E))
    lib().orc_returns(T, E, gamma, _dp(r), dn.ctypes.data_as(C.POINTER(C.c_ubyte)), _dp(vb), _dp(G))
    return G


def a2c_loss(logits, actions, adv, G, V, ent_coef: float, vf_coef: float):
    z = _f64(logits)
    S, A = z.shape
    a = np.ascontiguousarray(actions, dtype=np.int32).reshape(S)
    adv, G, V = _f64(adv).reshape(S), _f64(G).reshape(S), _f64(V).reshape(S)
    dz, dv, losses = np.empty((S, A)), np.empty(S), np.empty(4)
    lib().orc_a2c_loss(S, A, _dp(z), a.ctypes.data_as(C.POINTER(C.c_int)), _dp(adv), _dp(G), _dp(V),
                       ent_coef, vf_coef, _dp(dz), _dp(dv), _dp(losses))
    return dz, dv, losses


@dataclass
class HParams:
    """Table 2 defaults, except rms_eps/rms_alpha which the measured workloads fix."""
    lr: float = 7e-4
    rms_alpha: float = 0.99
    rms_eps: float = 1e-5
    gamma: float = 0.99
    ent_coef: float = 0.01
    vf_coef: float = 0.5
    max_grad_norm: float = 0.5      # <= 0: clipping off


def learner_grad(net: Net, params, rollout: dict, hp: HParams, workers: int = 1) -> dict:
    """Algorithm 1, returns/advantages and the A2C gradient for one agent.
    rollout: obs [T+1,E,...], actions [T,E], rewards [T,E], dones [T,E]."""
    obs = np.asarray(rollout["obs"])
    T1, E = obs.shape[0], obs.shape[1]
    T = T1 - 1
    flat = obs.reshape(T1 * E, -1)
    B = flat.shape[0]

    def chunks(n, k):
        k = max(1, min(k, n))
        b = [n * i // k for i in range(k + 1)]
        return [(b[i], b[i + 1]) for i in range(k) if b[i + 1] > b[i]]

    if workers > 1:
        with ThreadPoolExecutor(workers) as ex:
            outs = list(ex.map(lambda ab: forward(net, params, flat[ab[0]:ab[1]]), chunks(B, workers)))
        logits = np.concatenate([o[0] for o in outs])
        values = np.concatenate([o[1] for o in outs])
    else:
        logits, values = forward(net, params, flat)
    V = values.reshape(T1, E)
    G = returns(rollout["rewards"], rollout["dones"], V[T], hp.gamma)
    adv = G - V[:T]
    S = T * E
    dz, dv, losses = a2c_loss(logits[:S], np.asarray(rollout["actions"]).reshape(S), adv.reshape(S),
                              G.reshape(S), V[:T].reshape(S), hp.ent_coef, hp.vf_coef)
    if workers > 1:
        with ThreadPoolExecutor(workers) as ex:
            gs = list(ex.map(lambda ab: backward(net, params, flat[ab[0]:ab[1]], dz[ab[0]:ab[1]],
                                                 dv[ab[0]:ab[1]]), chunks(S, workers)))
        grad = np.sum(gs, axis=0)
    else:
        grad = backward(net, params, flat[:S], dz, dv)
    return dict(grad=grad, losses=losses, logits=logits, values=values, G=G, adv=adv,
                dlogits=dz, dvalues=dv)


# --------------------------------------------------------------------------
# optimiser
# --------------------------------------------------------------------------
def clip_coef(g, max_norm: float) -> Tuple[float, float]:
    """(c, ||g||_2) with c = min(1, max_norm/(||g||+1e-6)); max_norm<=0 -> c=1."""
    g = _f64(g).ravel()
    nrm = C.c_double()
    c = lib().orc_clip_coef(g.size, _dp(g), max_norm, C.byref(nrm))
    return float(c), float(nrm.value)


def rmsprop(x, g, v, clip: float, lr: float, alpha: float, eps: float):
    """Returns (y, v_new)."""
    x, g = _f64(x).ravel(), _f64(g).ravel()
    v2 = _f64(v).ravel().copy()
    y = np.empty_like(x)
    lib().orc_rmsprop(x.size, _dp(x), _dp(g), _dp(v2), clip, lr, alpha, eps, _dp(y))
    return y, v2


# --------------------------------------------------------------------------
# topology (integers only)
# --------------------------------------------------------------------------
RING, EXP, COMPLETE = 0, 1, 2


def in_peers(kind: int, peers: int, n: int, rnd: int, agent: int) -> List[int]:
    """In-peers of `agent` at round `rnd` (0-based agents).
    RING: directed ring v_0 -> v_1 -> ... -> v_{n-1} -> v_0 (Fig. 5): in-peers
      of i are i-1, ..., i-peers (mod n).
    EXP: time-varying exponential graph, L = ceil(log2 n); with p in-peers per
      round the j-th in-peer of i at round k is i - 2^((p*k + j) mod L) (mod n).
    COMPLETE: every other agent.
    Coinciding offsets are kept as separate terms (weights stay 1/(1+p))."""
    if n == 1:
        return []
    if kind == RING:
        return [(agent - o) % n for o in range(1, peers + 1)]
    if kind == EXP:
        L = max(1, (n - 1).bit_length())
        return [(agent - (1 << ((peers * rnd + j) % L))) % n for j in range(peers)]
    if kind == COMPLETE:
        return [j for j in range(n) if j != agent]
    raise ValueError(kind)


def mixing_matrix(kind: int, peers: int, n: int, rnd: int) -> np.ndarray:
    """Dense P^(k) with p_ij = 1/(1+|N_in_i|) (footnote of Algorithm 1)."""
    P = np.zeros((n, n))
    for i in range(n):
        nb = in_peers(kind, peers, n, rnd, i)
        w = 1.0 / (1 + len(nb))
        P[i, i] += w
        for j in nb:
            P[i, j] += w
    return P


def mix(own, msgs: Sequence[np.ndarray]) -> np.ndarray:
    own = _f64(own).ravel()
    ms = [_f64(m).ravel() for m in msgs]
    out = np.empty_like(own)
    arr = (C.POINTER(C.c_double) * max(1, len(ms)))(*[_dp(m) for m in ms])
    lib().orc_mix(own.size, _dp(own), len(ms), arr, _dp(out))
    return out


# --------------------------------------------------------------------------
# one gossip + optimiser pass over all agents
# --------------------------------------------------------------------------
def sweep_sync(X, G, V, hp: HParams, kind: int, peers: int, rnd: int,
               clips: Optional[Sequence[float]] = None):
    """Deterministic round, Eq. 7 with zero delay: every agent takes its
    RMSProp step, then all mix simultaneously with the peers' post-update,
    pre-mix parameters of the same round.  X, G, V: [n, d].
    Returns (X_new, V_new, Y) with Y the broadcast messages."""
    X, G, V = _f64(X), _f64(G), _f64(V)
    n = X.shape[0]
    Y, Vn = np.empty_like(X), np.empty_like(V)
    for i in range(n):
        c = clip_coef(G[i], hp.max_grad_norm)[0] if clips is None else clips[i]
        Y[i], Vn[i] = rmsprop(X[i], G[i], V[i], c, hp.lr, hp.rms_alpha, hp.rms_eps)
    Xn = np.empty_like(X)
    for i in range(n):
        Xn[i] = mix(Y[i], [Y[j] for j in in_peers(kind, peers, n, rnd, i)])
    return Xn, Vn, Y


def sweep_replay(x, g, v, hp: HParams, msgs: Optional[Sequence[np.ndarray]],
                 clip: Optional[float] = None):
    """One agent's asynchronous iteration (Algorithm 1; Eqs. 5-6): local step,
    then average with `msgs` if a fresh message from every in-peer was
    recorded, else keep the local result (msgs=None).  g=None: no pending
    gradient (publish + mix only).  Returns (x_new, v_new, y)."""
    if g is None:
        y, vn = _f64(x).ravel().copy(), _f64(v).ravel().copy()
    else:
        c = clip_coef(g, hp.max_grad_norm)[0] if clip is None else clip
        y, vn = rmsprop(x, g, v, c, hp.lr, hp.rms_alpha, hp.rms_eps)
    xn = y.copy() if msgs is None else mix(y, msgs)
    return xn, vn, y


def sync_round(net: Net, X, V, rollouts: Sequence[dict], hp: HParams, kind: int, peers: int,
               rnd: int, workers: int = 1):
    """One full synchronous round for all agents: learn, then sweep."""
    n = len(rollouts)
    if workers > 1:
        with ThreadPoolExecutor(workers) as ex:
            infos = list(ex.map(lambda i: learner_grad(net, X[i], rollouts[i], hp), range(n)))
    else:
        infos = [learner_grad(net, X[i], rollouts[i], hp) for i in range(n)]
    G = np.stack([f["grad"] for f in infos])
    Xn, Vn, Y = sweep_sync(X, G, V, hp, kind, peers, rnd)
    return Xn, Vn, infos


def consensus_distance(X) -> float:
    """||X - mean over agents||_F (Proposition 1)."""
    X = _f64(X)
    return float(np.linalg.norm(X - X.mean(axis=0, keepdims=True)))


def prop1_bound(update_norms: Sequence[float], betas) -> np.ndarray:
    """Right-hand side of Proposition 1 after rounds 0..K-1, for identical initial parameters:
        bound[k] = sum_{s=0..k} (prod_{r=s..k} beta_r) * ||alpha G(s)||_F ,
    update_norms[s] = ||alpha G(s)||_F (the step of round s, X - Y of that round), betas a scalar (the
    proposition's constant beta: bound[k] = alpha sum_s beta^(k+1-s) ||G(s)||) or one contraction factor per round
    (the second largest singular value of that round's doubly stochastic mixing matrix, which is what the proof's
    per-round inequality uses).  Written as the double sum of the statement, not as a recursion."""
    u = _f64(update_norms).ravel()
    K = u.size
    be = np.full(K, float(betas)) if np.ndim(betas) == 0 else _f64(betas).ravel()
    assert be.size == K
    out = np.zeros(K)
    for k in range(K):
        for s0 in range(k + 1):
            out[k] += np.prod(be[s0:k + 1]) * u[s0]
    return out


# --------------------------------------------------------------------------
# acting
# --------------------------------------------------------------------------
def sample(logits, u) -> np.ndarray:
    """Inverse-CDF draw per row: min{k : sum_{j<=k} pi_j > u}, clamped."""
    z = _f64(logits)
    u = _f64(u).ravel()
    out = np.empty(z.shape[0], dtype=np.int32)
    for s in range(z.shape[0]):
        out[s] = lib().orc_sample(z.shape[1], _dp(z[s]), float(u[s]))
    return out


def softmax(logits) -> np.ndarray:
    z = _f64(logits)
    z = z - z.max(axis=-1, keepdims=True)
    e = np.exp(z)
    return e / e.sum(axis=-1, keepdims=True)
