"""Shared helpers of the GPU parity tests: tolerance rule, oracle <-> library glue."""
from __future__ import annotations

import numpy as np

import gala_inputs as GI
from oracle import reference as R

# Tolerances (relative), one per arithmetic path.
TOL_SWEEP = 1e-5      # fp32 RMSProp + gossip pass fed identical fp32 inputs
TOL_FP32_NET = 1e-4   # fp32 network (MLP) outputs and gradients
TOL_BF16 = 2e-2       # bf16-operand GEMM outputs and gradients


def assert_close(name, got, want, tol, max_outliers=0):
    """Per tensor: ||a-b||_2 <= tol ||b||_2, and |a_i-b_i| <= tol (|b_i| + rms(b)) for every element but at most
    max_outliers of them.  max_outliers is 0 except where the caller has COUNTED, in the oracle alone, how many
    ReLU gates two valid evaluations of the same bf16 network disagree on (tie_allowance): a gate that falls the
    other way adds or removes one unit's whole contribution to a row of a weight gradient, which no tolerance on
    rounding covers.  Returns (relative l2 error, number of elements outside the bound)."""
    a = np.asarray(got, np.float64).ravel()
    b = np.asarray(want, np.float64).ravel()
    assert a.shape == b.shape, (name, a.shape, b.shape)
    assert np.isfinite(a).all(), name + ": non-finite values"
    nb = np.linalg.norm(b)
    rel = np.linalg.norm(a - b) / (nb if nb > 0 else 1.0)
    if not b.size:
        return rel, 0
    rms = nb / np.sqrt(b.size)
    ratio = np.abs(a - b) / (np.abs(b) + rms + 1e-30)
    inside = ratio <= tol
    outliers = int(b.size - inside.sum())
    # Without counted ties (max_outliers == 0) the l2 bound covers every element.  With them it covers the elements
    # inside the per-element bound, and a gross bound of 5 tol covers all: one gate of the hidden layer that falls
    # the other way for one of 80 samples moves 2 % of the l2 norm of every tensor below it (seen: one agent of
    # eight), which is the budgeted effect, not rounding.
    if max_outliers > 0:
        rel_in = np.linalg.norm((a - b)[inside]) / (nb if nb > 0 else 1.0)
        assert rel_in <= tol, "%s: relative l2 error of the elements inside the bound %.3e > %.1e" % (name, rel_in, tol)
        assert rel <= 5 * tol, "%s: relative l2 error %.3e > 5 x %.1e" % (name, rel, tol)
    else:
        assert rel <= tol, "%s: relative l2 error %.3e > %.1e" % (name, rel, tol)
    assert outliers <= max_outliers, "%s: %d elements beyond %.1e (|b_i| + rms b), %d allowed; worst %.3e (rel l2 %.3e)" % (
        name, outliers, tol, max_outliers, float(ratio.max()), rel)
    return rel, outliers


# Largest number of gradient elements that one ReLU gate can move beyond rounding: the unit's row of its own
# layer's weight gradient (3136 for the hidden layer, at most 576 for a convolution) plus what the changed dY
# does to the rows below through a 4x4 or 3x3 receptive field.
GATE_FAN_OUT = 4096


def tie_allowance(net: R.Net, params, obs) -> int:
    """Elements of a gradient that may lie outside the per-element bound, counted in the oracle alone: the number of
    ReLU gates on which two evaluations of the same bf16 network disagree - every sum formed exactly, and every sum
    formed in float32 term after term - plus one (a third evaluation, the GPU's, disagrees on gates of its own:
    about one in 10^6 units lies that close to zero, i.e. none to a few per test), times the fan-out of one gate.
    Nothing here comes from the GPU.  The test in which no gate CAN fall the other way (biases that fix every gate)
    allows no element at all."""
    if not net.bf16_operands:
        return 0
    from concurrent.futures import ThreadPoolExecutor
    o = np.asarray(obs).reshape(len(obs), -1)
    nl = len(net.convs) + len(net.hidden)
    f32 = net.with_f32_sums()

    def count(chunk):
        n = 0
        for li in range(nl):
            y0 = R.forward(net, params, chunk, which_layer=li)[2]
            y1 = R.forward(f32, params, chunk, which_layer=li)[2]
            n += int(((y0 > 0) != (y1 > 0)).sum())
        return n

    k = max(1, min(8, len(o) // 4))
    cuts = [len(o) * i // k for i in range(k + 1)]
    with ThreadPoolExecutor(k) as ex:
        flips = sum(ex.map(count, [o[cuts[i]:cuts[i + 1]] for i in range(k)]))
    return (flips + 1) * GATE_FAN_OUT


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


def assert_grad_close(name, got, want, net: R.Net, tol, max_outliers=0):
    """The tolerance rule applied per parameter tensor (conv1.W, conv1.b, ..., v.b); max_outliers is the budget
    of the whole gradient.  Returns the number of elements outside the per-element bound."""
    off = R.param_offsets(net)
    bounds = sorted((v, k) for k, v in off.items())
    total = 0
    for (lo, key), (hi, _) in zip(bounds[:-1], bounds[1:]):
        total += assert_close("%s/%s" % (name, key), np.asarray(got)[lo:hi], np.asarray(want)[lo:hi], tol,
                              max_outliers=max_outliers - total)[1]
    return total
