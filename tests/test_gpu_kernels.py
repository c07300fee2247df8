"""GPU parity: tensor-core GEMM entry point and the fused RMSProp + gossip pass,
each against the fp64 oracle / the plain definition, through the C ABI."""
import numpy as np
import pytest

import gala_inputs as GI
from oracle import reference as R
from tests.helpers import TOL_SWEEP, assert_close, to_bf16_f64

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def _B():
    from paper_1906_04585_b200 import binding
    return binding


# ---------------------------------------------------------------------- GEMM
GEMM_CASES = [
    # groups, M, N, K, a_mn, b_mn, split_k
    (1, 128, 128, 64, 0, 0, 1),
    (1, 128, 32, 256, 0, 0, 1),
    (2, 200, 64, 512, 0, 0, 1),       # ragged M, several groups
    (3, 300, 72, 136, 0, 0, 1),       # ragged M, N and K tails
    (1, 96, 512, 3136, 0, 0, 1),      # hidden layer forward shape
    (2, 80, 3136, 512, 0, 1, 1),      # data gradient of the hidden layer (B stored [K][N])
    (1, 392, 576, 64, 0, 1, 1),       # conv3 data gradient
    (2, 512, 3136, 80, 1, 1, 1),      # hidden layer weight gradient (both stored [K][.]), K tail
    (2, 576, 64, 3920, 1, 1, 4),      # conv3 weight gradient with split reduction
    (1, 256, 32, 6400, 1, 1, 7),      # conv1 weight gradient: N = 32 inside a 64-wide box
    (1, 256, 40, 200, 1, 0, 2),       # mixed: A stored [K][M], B stored [N][K]
    (1, 130, 130, 72, 0, 0, 3),       # more splits than K tiles
    (2, 300, 640, 200, 0, 0, 1),      # 256-column tiles (N >= 512): ragged M, N = 2.5 tiles, K tail
    (1, 264, 768, 520, 1, 0, 3),      # 256-column tiles with split reduction, A stored [K][M]
]


@pytest.mark.parametrize("case", GEMM_CASES)
def test_gemm_bf16_matches_definition(case):
    B = _B()
    groups, M, N, K, a_mn, b_mn, split = case
    rng = np.random.default_rng(hash(case) % (2 ** 31))
    a = rng.standard_normal((groups, M, K)).astype(np.float32)
    b = rng.standard_normal((groups, N, K)).astype(np.float32)
    a64, b64 = to_bf16_f64(a), to_bf16_f64(b)
    want = np.einsum("gmk,gnk->gmn", a64, b64)
    ta = torch.from_numpy(a).cuda().to(torch.bfloat16)
    tb = torch.from_numpy(b).cuda().to(torch.bfloat16)
    if a_mn:
        ta = ta.transpose(1, 2).contiguous()   # stored [K][M]
    if b_mn:
        tb = tb.transpose(1, 2).contiguous()   # stored [K][N]
    td = torch.full((groups, M, N), float("nan"), device="cuda", dtype=torch.float32)
    B.gala_gemm_bf16(ta, tb, td, groups, M, N, K, a_mn, b_mn, split, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    # exact bf16 products accumulated in fp32 on the tensor cores (K up to 6400 terms)
    assert_close("D", td.cpu().numpy(), want, 1e-4)


# --------------------------------------------------------------------- sweep
def _sweep_case(n, d, kind, peers, rounds, clip, seed):
    B = _B()
    x, g, v = GI.sweep_state(n, d, seed)
    d_pad = (d + 3) // 4 * 4
    hp = B.default_hparams(1, 1, max_grad_norm=0.0)
    ohp = R.HParams(lr=float(hp.lr), rms_alpha=float(hp.rms_alpha), rms_eps=float(hp.rms_eps), max_grad_norm=0.0)
    topo = B.gala_topology(kind, peers)

    def pad(a):
        out = np.zeros((n, d_pad), np.float32)
        out[:, :d] = a
        return out

    tx, tg, tv = (torch.from_numpy(pad(t)).cuda() for t in (x, g, v))
    clips = None
    tclip = None
    if clip:
        clips = (0.25 + 0.75 * np.random.default_rng(seed).random(n)).astype(np.float32)
        tclip = torch.from_numpy(clips).cuda()
    X, V = x.astype(np.float64), v.astype(np.float64)
    for k in range(rounds):
        B.gala_sweep_sync(tx, tg, tv, tclip, n, d_pad, topo, k, hp, torch.cuda.current_stream().cuda_stream)
        X, V, _ = R.sweep_sync(X, g, V, ohp, kind, peers, k, clips=None if clips is None else [float(c) for c in clips])
    torch.cuda.synchronize()
    assert_close("x", tx.cpu().numpy()[:, :d], X, TOL_SWEEP)
    assert_close("v", tv.cpu().numpy()[:, :d], V, TOL_SWEEP)


@pytest.mark.parametrize("n,kind,peers", [(4, R.RING, 1), (8, R.EXP, 1), (32, R.EXP, 1), (32, R.EXP, 2),
                                          (5, R.EXP, 2), (3, R.RING, 2), (64, R.EXP, 1), (1, R.RING, 1)])
def test_sweep_sync_matches_oracle(n, kind, peers):
    # ragged length (not a multiple of the tile), several rounds of the time-varying schedule
    _sweep_case(n, 10_007, kind, peers, rounds=4, clip=(n % 2 == 0), seed=GI.BASE_SEED + 3)


def test_sweep_sync_full_size_sampled():
    # the micro-benchmark's size (32 agents x 1.7M parameters); the oracle recomputes a sample of
    # columns, which is exact because the pass is element-wise across the parameter index.
    B = _B()
    w = GI.WORKLOADS[3]
    n, d = w.n_agents, w.sweep_only_d
    x, g, v = GI.sweep_state(n, d, w.seed)
    hp = B.default_hparams(1, 1, max_grad_norm=0.0)
    ohp = R.HParams(lr=float(hp.lr), rms_alpha=float(hp.rms_alpha), rms_eps=float(hp.rms_eps), max_grad_norm=0.0)
    rng = np.random.default_rng(7)
    cols = np.unique(np.concatenate([np.arange(2048), np.arange(d - 2048, d), rng.integers(0, d, 20000)]))
    for peers in (1, 2):
        topo = B.gala_topology(B.GALA_TOPO_EXP, peers)
        tx, tg, tv = (torch.from_numpy(t).cuda() for t in (x, g, v))
        X, V = x[:, cols].astype(np.float64), v[:, cols].astype(np.float64)
        for k in range(3):
            B.gala_sweep_sync(tx, tg, tv, None, n, d, topo, k, hp, torch.cuda.current_stream().cuda_stream)
            X, V, _ = R.sweep_sync(X, g[:, cols], V, ohp, R.EXP, peers, k, clips=[1.0] * n)
        torch.cuda.synchronize()
        assert_close("x", tx.cpu().numpy()[:, cols], X, TOL_SWEEP)
        assert_close("v", tv.cpu().numpy()[:, cols], V, TOL_SWEEP)
        # invariant at any size: the exponential schedule is doubly stochastic, so with zero
        # gradients the column mean is preserved
        tz = torch.zeros_like(tg)
        before = tx.double().mean(dim=0)
        B.gala_sweep_sync(tx, tz, tv, None, n, d, topo, 5, hp, torch.cuda.current_stream().cuda_stream)
        after = tx.double().mean(dim=0)
        assert float((after - before).abs().max()) < 1e-8
