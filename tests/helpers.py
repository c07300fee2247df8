"""Shared helpers of the GPU parity tests: tolerance rule, oracle <-> library glue."""
from __future__ import annotations

import numpy as np

import gala_inputs as GI
from oracle import reference as R

# Tolerances (relative), one per arithmetic path.
TOL_SWEEP = 1e-5      # fp32 RMSProp + gossip pass fed identical fp32 inputs
TOL_FP32_NET = 1e-4   # fp32 network (MLP) outputs and gradients
TOL_BF16 = 2e-2       # bf16-operand GEMM outputs and gradients


def assert_close(name, got, want, tol, rule="elementwise"):
    """Per tensor.  Both rules demand ||a-b||_2 <= tol ||b||_2.
    rule "elementwise" (fp32 paths) adds |a_i-b_i| <= tol (|b_i| + rms(b)) for every element.
    rule "norm" (bf16-operand paths) adds max|a_i-b_i| <= 5 tol max|b_i| instead.  Two things make a
    per-element bound relative to rms(b) meaningless there: a stored bf16 operand that lands one unit
    in the last place apart on the two sides (fp32 vs exact summation next to a rounding boundary) moves
    a single product by 0.4 %; and a ReLU input within fp32 summation noise of zero may fall on either
    side of the gate, which adds or removes that unit's whole contribution (one row of a weight
    gradient for one sample).  With millions of gated units per step a few such ties are expected; they
    stay far below tol in l2 but can reach a few % of max|b| on single elements."""
    a = np.asarray(got, np.float64).ravel()
    b = np.asarray(want, np.float64).ravel()
    assert a.shape == b.shape, (name, a.shape, b.shape)
    assert np.isfinite(a).all(), name + ": non-finite values"
    nb = np.linalg.norm(b)
    rel = np.linalg.norm(a - b) / (nb if nb > 0 else 1.0)
    assert rel <= tol, "%s: relative l2 error %.3e > %.1e" % (name, rel, tol)
    if not b.size:
        return rel
    if rule == "elementwise":
        rms = nb / np.sqrt(b.size)
        worst = np.max(np.abs(a - b) / (np.abs(b) + rms + 1e-30))
    else:
        worst = np.max(np.abs(a - b)) / (np.max(np.abs(b)) + 1e-30) / 5.0
    assert worst <= tol, "%s: worst element error %.3e > %.1e (rel l2 %.3e, rule %s)" % (name, worst, tol, rel, rule)
    return rel


def oracle_net(w: GI.Workload, exact: bool = False) -> R.Net:
    """The oracle's network for a workload.  The conv workloads are specified with bf16 GEMM
    operands, so their oracle rounds the contraction operands to bf16 (exact sums); `exact`
    asks for the unrounded fp64 network instead."""
    if w.net_kind == "conv":
        return R.Net.atari(w.n_actions).with_bf16(not exact)
    return R.Net.mlp(w.obs_dim, w.hidden, w.n_actions)


def oracle_hp(hp) -> R.HParams:
    """Oracle hyper-parameters = the float32 values the library was given, widened."""
    return R.HParams(lr=float(hp.lr), rms_alpha=float(hp.rms_alpha), rms_eps=float(hp.rms_eps),
                     gamma=float(hp.gamma), ent_coef=float(hp.ent_coef), vf_coef=float(hp.vf_coef),
                     max_grad_norm=float(hp.max_grad_norm))


def to_bf16_f64(a: np.ndarray) -> np.ndarray:
    """Round float32 values to bfloat16 (nearest even) and return them as float64."""
    u = np.ascontiguousarray(a, np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64)


def assert_grad_close(name, got, want, net: R.Net, tol, rule="elementwise"):
    """The tolerance rule applied per parameter tensor (conv1.W, conv1.b, ..., v.b)."""
    off = R.param_offsets(net)
    bounds = sorted((v, k) for k, v in off.items())
    for (lo, key), (hi, _) in zip(bounds[:-1], bounds[1:]):
        assert_close("%s/%s" % (name, key), np.asarray(got)[lo:hi], np.asarray(want)[lo:hi], tol, rule)
