#!/usr/bin/env python
"""Throughput of the GALA-A2C learner step on B200.

One "step" is one pass of the whole learner path for all agents of a workload:
network forward/backward over each agent's rollout, returns / advantages / A2C
objective, global-norm clip, and the fused RMSProp + gossip pass.

  python bench.py [--gpus N --steps K --warmup W]            the CUDA library
  python bench.py --impl reference [...]                     the fp64 CPU oracle

With no --workload the line's headline is the largest workload in its stated
mode - 64 agents, conv net, asynchronous: every agent's rollout arrives after a
random simulator delay and whatever has arrived goes to the learner as one
grouped call - and the other workloads (64 and 16 agents synchronous, the same
64 agents in a synchronous loop that waits for the slowest simulator, 8 agents,
the small MLP) follow as named sub-records under "workloads", each with its own
step time, dominant-kernel roofline, whole-round roofline and end-to-end rate.
The fused RMSProp + gossip pass alone (32 agents x 1.7 M parameters) is timed
in its all-agent and per-agent forms under "sweep_microbench".

Prints one JSON line on rank 0.  With N > 1 (torchrun) every rank runs an
independent replica of the workload on its own GPU (the path has no
cross-GPU exchange); the value is the sum over ranks over the slowest rank's
time.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import gala_inputs as GI  # noqa: E402

METRIC = "learner frames/s for N agents on 1 B200"
UNIT = "frames/s"
L2_BYTES = 126 * 1024 * 1024
MIN_REGION_S = 0.3           # every timed region lasts at least this long (the step list is repeated)

# dram__bytes_read.sum + dram__bytes_write.sum per launch from an ncu capture of the kernel class named, on the
# workload named, taken on the kernels as they are now; an entry is removed when its kernel changes.
NCU_TRAFFIC_BYTES = {
    # all-agent optimiser / gossip pass inside the c2 round (kernel unchanged since the capture): 162.1 MB read +
    # 78.4 MB written against 297.2 MB algorithmic; part of the output is still in L2 when the kernel ends
    ("c2_conv_exp_n8", "sweep_sync"): 240.5e6,
    # conv1 forward at c3: 304.2 MB read (the uint8 frames, once) + 250.3 MB written (act1 and gate words)
    ("c3_conv_exp_n16", "gemm_conv1_fwd"): 554.5e6,
}
# For classes whose launches differ in size (the grouped optimiser / gossip pass takes the agents that were ready):
# dram bytes / algorithmic bytes from an ncu capture of the same kernel (32 agents x 1.7 M parameters, every agent
# averaging with one in-peer: 1 472.9 MB against 1 523.2 MB); its traffic is proportional to agents x parameters.
NCU_TRAFFIC_RATIO = {"sweep_agent": 1472.9 / 1523.2}


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm=float(p["hbm_gbs"]), tensor=float(p["bf16_tflops_sustained"]), source="measured")
    return dict(hbm=6650.0, tensor=1400.0, source="fallback")


# ----------------------------------------------------------------------------- work per class
def class_work(w: GI.Workload, d_pad: int):
    """Algorithmic work of one step per kernel class: name -> (bound, amount), amount in bytes
    (hbm) or flops (tensor), summed over the launches of that class in one step."""
    n, E, T, A = w.n_agents, w.n_envs, w.n_steps, w.n_actions
    B, S = (T + 1) * E, T * E
    shadow = 2.0 if w.net_kind == "conv" else 0.0
    out = {"sweep_sync": ("hbm", n * d_pad * (20.0 + shadow)),
           # per-agent form: read x, g, v and p snapshots, write x, v and the own snapshot (every agent averaging)
           "sweep_agent": ("hbm", n * d_pad * (24.0 + 4.0 * w.topo_peers + shadow)),
           # the conv net's norm pass skips the hidden layer's weight gradient (its sums of squares come with it)
           "grad_norm": ("hbm", n * (d_pad - (512 * 3136 if w.net_kind == "conv" else 0)) * 4.0)}
    if w.net_kind != "conv":
        return out
    P, KK, CO = (400, 81, 49), (256, 512, 576), (32, 64, 64)
    out["cast_frames"] = ("hbm", n * B * (84 * 84 * 4 * 3.0))      # uint8 in, bf16 out
    for l in range(3):
        out["gemm_conv%d_fwd" % (l + 1)] = ("tensor", 2.0 * n * B * P[l] * KK[l] * CO[l])
        out["gemm_conv%d_wgrad" % (l + 1)] = ("tensor", 2.0 * n * S * P[l] * KK[l] * CO[l])
        if l > 0:
            out["gemm_conv%d_dgrad" % (l + 1)] = ("tensor", 2.0 * n * S * P[l] * KK[l] * CO[l])
    out["gemm_fc_fwd"] = ("tensor", 2.0 * n * B * 3136 * 512)
    out["gemm_fc_wgrad"] = ("tensor", 2.0 * n * S * 3136 * 512)
    out["gemm_fc_dgrad"] = ("tensor", 2.0 * n * S * 3136 * 512)
    out["colsum"] = ("hbm", n * S * (512 + 49 * 64 + 81 * 64 + 400 * 32) * 2.0)
    return out


def round_work(w: GI.Workload, d_pad: int, per_agent_sweep: bool = False):
    """Algorithmic HBM bytes and tensor flops of one whole round with the tensors this build keeps in memory
    (every stored tensor written once and read once per kernel that consumes it; nothing lowered)."""
    n, E, T = w.n_agents, w.n_envs, w.n_steps
    B, S = (T + 1) * E, T * E
    sweep = (24.0 + 4.0 * w.topo_peers) if per_agent_sweep else 20.0
    if w.net_kind != "conv":
        return n * d_pad * (sweep + 4.0), 0.0
    act = (400 * 32, 81 * 64, 49 * 64)                     # elements per sample of act1..3
    by = B * 84 * 84 * 4 + S * 84 * 84 * 4                 # uint8 frames: forward, conv1 weight gradient
    for a in act:
        by += B * a * 2 + B * a * 2 + S * a * 2            # activation written, read forward, read by a weight gradient
        by += B * a / 8 + S * a / 8                        # ReLU gate bits written and read
        # dY: written, read by the weight gradient (which also sums conv2's / conv3's bias gradient) and, except
        # for conv1, by the data gradient; dY1 is read once more by the column sums only in small launches
        # (larger ones take conv1's bias gradient out of conv2's data gradient)
        by += S * a * 2 * (3 if a != act[0] else (3 if n * S < 2048 else 2))
    by += B * 512 * 2 * 2 + S * 512 * 2                    # hidden activations: written, read by heads, read by head gradients
    by += S * 512 * 2 * 4                                  # dh: written, read by FC data / weight gradient and bias sums
    by += 2 * (d_pad * 2) + d_pad * 4 + d_pad * 4          # bf16 weights forward + backward, gradient written, read by the norm
    by += d_pad * (sweep + 2.0)                            # optimiser / gossip pass with the bf16 copy
    P, KK, CO = (400, 81, 49), (256, 512, 576), (32, 64, 64)
    fl = 0.0
    for l in range(3):
        fl += 2.0 * P[l] * KK[l] * CO[l] * (B + S + (S if l > 0 else 0))
    fl += 2.0 * 3136 * 512 * (B + 2 * S)
    return n * by, n * fl


# ----------------------------------------------------------------------------- ranks
def max_over_ranks(x: float, device: str = "cuda") -> float:
    """The slowest rank's value (every rank gets it); the local value when there is one process.  The agents of
    one rank never talk to those of another (replicas only), so this is the only collective of a multi-rank run."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([x], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(frames_per_rank: float, local_seconds: float, world: int, device: str = "cuda") -> float:
    """Frames/s of the whole job: all ranks' frames over the slowest rank's time."""
    return frames_per_rank * world / max_over_ranks(local_seconds, device)


def median(xs) -> float:
    return float(np.median(np.asarray(xs, dtype=np.float64)))


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """nvidia-smi samples every 20 ms for the whole run; window() summarises those inside a time span."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.proc = None
        self.gpu = gpu_index
        self.rows = None
        # samples go to a scratch file (BENCH_CLOCKS_DIR, else the system's temporary directory); the line that is
        # printed carries their summary
        import tempfile
        self.path = os.path.join(os.environ.get("BENCH_CLOCKS_DIR", tempfile.gettempdir()),
                                 "bench_clocks_%d.csv" % os.getpid())

    def start(self):
        try:
            os.makedirs(os.path.dirname(self.path), exist_ok=True)
            self.f = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        import datetime
        self.rows = []
        if self.proc is None:
            return
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.close()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in open(self.path):
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                self.rows.append((ts, float(parts[1]), float(parts[2]),
                                  [nm for nm, val in zip(names, parts[5:9]) if val.lower().startswith("active")]))
            except ValueError:
                continue

    def window(self, t_begin: float, t_end: float):
        """Median SM clock and throttle reasons over the samples taken inside [t_begin, t_end] (time.time()
        values); if the span held no sample, over the samples nearest to it."""
        out = dict(sm_mhz=None, sm_max_mhz=None, reasons=[], samples=0)
        rows = self.rows or []
        inside = [r for r in rows if t_begin - 0.02 <= r[0] <= t_end + 0.02]
        if not inside and rows:
            mid = 0.5 * (t_begin + t_end)
            inside = sorted(rows, key=lambda r: abs(r[0] - mid))[:3]
        if inside:
            out = dict(sm_mhz=float(np.median([r[1] for r in inside])), sm_max_mhz=float(max(r[2] for r in inside)),
                       reasons=sorted({nm for r in inside for nm in r[3]}), samples=len(inside))
        return out


# ----------------------------------------------------------------------------- CPU oracle legs
def oracle_sample_rate(w: GI.Workload, n_envs: int, workers: int, agents: int = 1):
    """Frames/s of the oracle on `agents` agents' rollouts cut down to n_envs environments (learner
    step + optimiser/gossip pass per agent).  Returns (frames_per_s, seconds)."""
    from oracle import reference as R
    net = R.Net.atari(w.n_actions).with_bf16() if w.net_kind == "conv" else R.Net.mlp(w.obs_dim, w.hidden, w.n_actions)
    hp = R.HParams()
    ws = w.scaled(n_envs=n_envs)
    p0 = GI.init_params(GI.net_tensors(w), w.seed).astype(np.float64)
    v0 = np.zeros_like(p0)
    ros = [GI.rollout(ws, i, 0) for i in range(agents)]
    t0 = time.perf_counter()
    for ro in ros:
        info = R.learner_grad(net, p0, ro, hp, workers=workers)
        R.sweep_replay(p0, info["grad"], v0, hp, [p0])
    dt = time.perf_counter() - t0
    return agents * n_envs * w.n_steps / dt, dt


def usable_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def cpu_baseline(w: GI.Workload, budget_s: float = 12.0):
    """The oracle as it stands on a bounded sample of the workload: once on all cores it may use (at most 16
    worker threads) and once on one thread, each sized from a one-environment calibration to about budget_s."""
    cores = usable_cores()
    workers = min(cores, 16)
    _, t1 = oracle_sample_rate(w, 1, 1)                      # one agent, one environment, one thread
    per_env_1 = max(t1, 1e-3)
    e1 = int(max(1, min(w.n_envs, budget_s / per_env_1)))
    v1, dt1 = oracle_sample_rate(w, e1, 1)
    per_env_m = per_env_1 / max(1.0, 0.6 * workers)          # rough: the threads split the samples
    tot = budget_s / per_env_m                               # environments that fit the budget
    agents = int(max(1, min(w.n_agents, tot // w.n_envs)))
    em = w.n_envs if tot >= w.n_envs else int(max(1, tot))
    vm, dtm = oracle_sample_rate(w, em, workers, agents=agents)
    return dict(value=vm, unit=UNIT, cores=workers, kind="oracle",
                sample="%d of %d agents x (%d of %d envs x %d steps), learner step + optimiser/gossip pass per agent, "
                       "%.1f s" % (agents, w.n_agents, em, w.n_envs, w.n_steps, dtm),
                one_thread=dict(value=v1, cores=1, sample="1 agent x (%d of %d envs x %d steps), %.1f s"
                                                           % (e1, w.n_envs, w.n_steps, dt1)))


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = GI.WORKLOADS[args.workload if args.workload >= 0 else 4]
    cores = usable_cores()
    workers = min(cores, 16)
    _, t1 = oracle_sample_rate(w, 1, workers)                 # calibration on one environment
    budget = 150.0 / max(1, args.steps + args.warmup)
    n_envs = int(max(1, min(w.n_envs, budget / max(t1, 1e-3))))
    for _ in range(args.warmup):
        oracle_sample_rate(w, n_envs, workers)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_sample_rate(w, n_envs, workers)
    dt = time.perf_counter() - t0
    value = args.steps * n_envs * w.n_steps / dt
    sample = "per step: 1 of %d agents, %d of %d envs x %d steps, learner step + optimiser/gossip pass" % (
        w.n_agents, n_envs, w.n_envs, w.n_steps)
    line = dict(impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps,
                warmup=args.warmup, ms_per_step=1e3 * dt / args.steps, higher_is_better=True, scaling="weak",
                vs_baseline=None, dtype="f64", data="synthetic",
                config=dict(workload=w.name, sample=sample),
                cpu_baseline=dict(value=value, unit=UNIT, cores=workers, kind="oracle", sample=sample),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))


# ----------------------------------------------------------------------------- the CUDA library
class Env:
    """What every measurement shares: modules, rank layout, peaks, the L2 flush buffer."""

    def __init__(self, args):
        import torch
        import torch.distributed as dist
        from paper_1906_04585_b200 import binding as B
        from paper_1906_04585_b200 import learner as LM
        self.torch, self.dist, self.B, self.LM, self.args = torch, dist, B, LM, args
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        torch.cuda.set_device(self.local)
        if self.world > 1:
            dist.init_process_group("nccl", device_id=torch.device("cuda", self.local))
        self.pk = peaks()
        self.flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device="cuda")
        self.spans = []          # (key, time.time() at begin, at end) of every timed region
        self.sets = {}           # workload index -> its rollout buffer sets (one workload at a time)

    def barrier(self):
        if self.world > 1:
            self.dist.barrier()
        self.torch.cuda.synchronize()


def spin_until(t: float):
    while time.perf_counter() < t:
        pass


def measure(env: Env, w: GI.Workload, mode: str, key: str, e2e: bool = True):
    """One workload in one mode.
    mode "sync": synchronous all-agent rounds (gala_step_sync), device time per round from events.
         "sync_stragglers": the same rounds, each started only when the slowest of the agents' simulator delays
                   ~Exp(mean one solo agent step) has passed since the previous round ended (host clock).
         "async": every agent's next rollout arrives a delay ~Exp(same mean) after its previous iteration
                   completed on the device; a host loop hands whatever has arrived to gala_learn_many /
                   gala_gossip_many while at most two such calls are in flight (host clock).
         "async_noskew": no delays: every round all agents in random order as one grouped call, rounds enqueued
                   back to back (host clock between two waits).
    """
    torch, B, LM, args = env.torch, env.B, env.LM, env.args
    world, rank = env.world, env.rank
    n = w.n_agents
    L = LM.Learner(n, w.topo_kind, w.topo_peers, w.net_kind, w.n_actions, w.n_envs, w.n_steps,
                   obs_dim=w.obs_dim, hidden=w.hidden)
    p0 = GI.init_params(GI.net_tensors(w), w.seed)
    for i in range(n):
        L.set_state(i, params=p0, sq_avg=np.zeros(L.d, np.float32))
    if args.no_graphs:
        B.gala_set_graphs(L.ctx, False)
    if args.lanes:
        B.gala_set_group_lanes(L.ctx, args.lanes)
    ext = torch.cuda.ExternalStream(B.gala_get_stream(L.ctx, -1))
    up = torch.cuda.Stream()      # host -> device copies run on a torch stream; the library's stream waits on it
    n_sets = 4
    # a round's rollouts of all agents share one pinned host buffer and one device buffer per field; the sets of a
    # workload are generated once and serve all its modes
    if w.index not in env.sets:
        env.sets.clear()
        env.sets[w.index] = [LM.RolloutBatch([GI.rollout(w, i, s + 1000 * rank) for i in range(n)]) for s in range(n_sets)]
    sets = env.sets[w.index]
    n_classes = B.gala_kernel_classes()
    names = [B.gala_kernel_class_name(k) for k in range(n_classes)]
    work = class_work(w, L.d_pad)
    is_async = mode in ("async", "async_noskew")
    rng = np.random.default_rng(w.seed)
    K = args.steps
    frames_per_step = w.frames_per_round

    # ------------------------------------------------------------------ step drivers
    def sync_step(cur):
        L.step_sync(cur)

    def grouped_round(cur):
        order = [int(i) for i in rng.permutation(n)]
        L.learn_many(order, [cur[i] for i in order])
        L.gossip_many(order)

    iters = np.zeros(n, dtype=np.int64)

    def async_region(steps: int, mean_s: float):
        """steps * n agent iterations with simulator delays; returns the host seconds it took."""
        target = steps * n
        busy = np.zeros(n, dtype=bool)
        t0 = time.perf_counter()
        ready_at = t0 + rng.exponential(mean_s, n)
        inflight = []                              # (an agent of the call, its members), oldest first
        done = launched = 0
        thresh = max(1, n // 2)
        sizes = []
        while done < target:
            while inflight and not B.gala_poll_agent(L.ctx, inflight[0][0]):
                _, members = inflight.pop(0)
                now = time.perf_counter()
                busy[members] = False
                ready_at[members] = now + rng.exponential(mean_s, len(members))
                done += len(members)
            if launched < target and len(inflight) < 2:
                now = time.perf_counter()
                R = np.nonzero(~busy & (ready_at <= now))[0]
                if len(R) and (not inflight or len(R) >= thresh):
                    lst = [int(i) for i in R[:target - launched]]
                    L.learn_many(lst, [sets[int(iters[i]) % n_sets][i] for i in lst])
                    L.gossip_many(lst)
                    busy[lst] = True
                    iters[lst] += 1
                    launched += len(lst)
                    inflight.append((lst[-1], lst))
                    sizes.append(len(lst))
        L.sync()
        return time.perf_counter() - t0, sizes

    def straggler_region(steps: int, mean_s: float):
        """steps synchronous rounds, each waiting for the slowest of n simulator delays first."""
        t0 = time.perf_counter()
        t_done = t0
        for k in range(steps):
            spin_until(t_done + float(rng.exponential(mean_s, n).max()))
            L.step_sync(sets[k % n_sets])
            L.sync()
            t_done = time.perf_counter()
        return t_done - t0

    # ------------------------------------------------------------------ simulator delay: one agent's own step time
    mean_delay_s = 0.0
    if mode in ("async", "sync_stragglers"):
        for _ in range(3):
            L.learn_many([0], [sets[0][0]]); L.gossip_many([0])
        L.sync()
        t0 = time.perf_counter()
        for _ in range(10):
            L.learn_many([0], [sets[0][0]]); L.gossip_many([0])
        L.sync()
        mean_delay_s = (time.perf_counter() - t0) / 10

    def run_steps(steps: int):
        """Untimed helper for warm-up: `steps` steps of this mode."""
        if mode == "sync":
            for k in range(steps):
                sync_step(sets[k % n_sets])
        elif mode == "async_noskew":
            for k in range(steps):
                grouped_round(sets[k % n_sets])
        elif mode == "async":
            async_region(steps, mean_delay_s)
        else:
            straggler_region(steps, mean_delay_s)
        L.sync()

    # warm-up; two steps first (lazy module loading lands on whichever kernel runs first), then steps that time
    # every kernel class to find the dominant one
    run_steps(2)
    B.gala_profile_enable(L.ctx, (1 << n_classes) - 1)
    wsteps = max(3, args.warmup)
    run_steps(wsteps)
    prof_all = B.gala_profile_read(L.ctx, reset=True)
    per_class_ms = {k: v[0] / wsteps for k, v in prof_all.items() if v[1] > 0}
    dominant = max(per_class_ms, key=per_class_ms.get)
    if dominant not in work:
        # small fp32 kernels of the MLP workload: neither bandwidth nor arithmetic bounds them (5 061 parameters and
        # 80 samples per agent), a launch is a few microseconds of latency; the optimiser pass is reported instead
        dominant = "sweep_agent" if is_async else "sweep_sync"
    B.gala_profile_enable(L.ctx, 1 << names.index(dominant))
    # estimate of a step, to size the timed region
    t0 = time.perf_counter()
    run_steps(2)
    est = max(1e-5, (time.perf_counter() - t0) / 2)
    B.gala_profile_read(L.ctx, reset=True)
    reps = max(1, int(math.ceil(MIN_REGION_S / (est * K))))
    total_steps = reps * K

    # ------------------------------------------------------------------ timed region
    st0 = [B.gala_stats(L.ctx, i) for i in range(n)] if is_async else None
    env.barrier()
    launches0 = L.launches()
    t_clock0 = time.time()
    t_wall0 = time.perf_counter()
    block_ms = []
    group_sizes = []
    if mode == "sync":
        # device time per step from events on the launching stream, L2 flushed between steps (outside the pairs)
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(total_steps)]
        for k in range(total_steps):
            with torch.cuda.stream(ext):
                env.flush.zero_()
            ev[k][0].record(ext)
            sync_step(sets[k % n_sets])
            ev[k][1].record(ext)
        L.sync()
        step_ms = [a.elapsed_time(b) for a, b in ev]
    else:
        # host clock between two waits, one block of K steps at a time; a round's inputs (0.7 GB of frames at 64
        # agents) are far larger than L2, so nothing is flushed
        step_ms = []
        for r in range(reps):
            if mode == "async_noskew":
                t0 = time.perf_counter()
                for k in range(K):
                    grouped_round(sets[k % n_sets])
                L.sync()
                dt = time.perf_counter() - t0
            elif mode == "async":
                dt, sizes = async_region(K, mean_delay_s)
                group_sizes += sizes
            else:
                dt = straggler_region(K, mean_delay_s)
            step_ms += [1e3 * dt / K] * K
            block_ms.append(1e3 * dt / K)
    env.barrier()
    t_wall = time.perf_counter() - t_wall0
    t_clock1 = time.time()
    env.spans.append((key, t_clock0, t_clock1))
    launches = L.launches() - launches0
    prof = B.gala_profile_read(L.ctx, reset=True)
    B.gala_profile_enable(L.ctx, 0)
    med_ms = max_over_ranks(median(step_ms))
    mean_ms = max_over_ranks(float(np.mean(step_ms)))
    value = frames_per_step * world / (med_ms * 1e-3)

    # ------------------------------------------------------------------ roofline of the dominant kernel class
    pk = env.pk
    dom_ms, dom_timed, _ = prof[dominant]
    bound, amount = work.get(dominant, ("hbm", 0.0))
    mixes = skipped = 0
    mixed_frac = None
    st1 = None
    if is_async:
        st1 = [B.gala_stats(L.ctx, i) for i in range(n)]
        mixes = sum(b["mixes"] - a["mixes"] for a, b in zip(st0, st1))
        skipped = sum(b["skipped"] - a["skipped"] for a, b in zip(st0, st1))
        mixed_frac = mixes / max(1, mixes + skipped)
        if dominant == "sweep_agent":    # only the steps that averaged read their in-peers' snapshots
            amount = n * L.d_pad * (24.0 + 4.0 * w.topo_peers * mixed_frac + (2.0 if w.net_kind == "conv" else 0.0))
    per_step_ms = dom_ms / max(1, total_steps)
    per_launch_ms = dom_ms / max(1, dom_timed)
    launches_per_step = dom_timed / max(1, total_steps)
    if bound == "hbm":
        achieved = amount / (per_step_ms * 1e-3) / 1e9 if per_step_ms > 0 else 0.0
        peak, unit = pk["hbm"], "GB/s"
    else:
        achieved = amount / (per_step_ms * 1e-3) / 1e12 if per_step_ms > 0 else 0.0
        peak, unit = pk["tensor"], "TFLOP/s"
    traffic = NCU_TRAFFIC_BYTES.get((w.name, dominant))
    if traffic is None and dominant in NCU_TRAFFIC_RATIO and launches_per_step > 0:
        traffic = NCU_TRAFFIC_RATIO[dominant] * amount / launches_per_step   # per launch, like `achieved`
    roofline = dict(kernel=dominant, bound=bound, achieved=achieved, peak=peak, unit=unit, frac=achieved / peak,
                    peak_source=pk["source"], traffic=traffic,
                    algorithmic_per_step=amount, ms_per_step=per_step_ms, ms_per_launch=per_launch_ms,
                    launches_per_step=launches_per_step, launches_timed=int(dom_timed),
                    share_of_step=per_step_ms / med_ms if med_ms > 0 else None)
    if bound == "hbm":
        roofline["frac_of_8tbs"] = achieved / 8000.0
        if traffic:   # the same launch by the bytes that crossed DRAM (part of the rest was served by L2)
            roofline["dram_gbs"] = traffic / (per_launch_ms * 1e-3) / 1e9
            roofline["frac_dram"] = roofline["dram_gbs"] / peak

    rb, rf = round_work(w, L.d_pad, per_agent_sweep=is_async)
    t_hbm, t_tensor = rb / (pk["hbm"] * 1e9) * 1e3, rf / (pk["tensor"] * 1e12) * 1e3
    round_roofline = dict(hbm_bytes=rb, tensor_flops=rf, hbm_ms=t_hbm, tensor_ms=t_tensor,
                          bound="hbm" if t_hbm >= t_tensor else "tensor",
                          frac=max(t_hbm, t_tensor) / med_ms if med_ms > 0 else None,
                          note="whole round against min-time at the measured copy bandwidth / sustained bf16 rate")
    mode_text = {
        "sync": "synchronous round (gala_step_sync), device time per round from CUDA events",
        "sync_stragglers": "synchronous rounds, each started when the slowest of the agents' simulator delays "
                           "~Exp(mean %d us) has passed since the previous round ended; host clock" % (mean_delay_s * 1e6),
        "async": "asynchronous: an agent's rollout arrives ~Exp(mean %d us = one solo agent step) after its previous "
                 "iteration completed; arrived agents go to gala_learn_many + gala_gossip_many, at most two calls "
                 "in flight; host clock" % (mean_delay_s * 1e6),
        "async_noskew": "asynchronous calls without simulator delays: each round all agents in random order as one "
                        "gala_learn_many + gala_gossip_many, rounds enqueued back to back; host clock",
    }[mode]
    topo_name = ("exp%d" if w.topo_kind == GI.EXP else "ring%d") % w.topo_peers
    rec = dict(workload=w.name, mode=mode, value=value, unit=UNIT, ms_per_step=med_ms, ms_per_step_mean=mean_ms,
               timed_steps=total_steps, frames_per_step=frames_per_step, gpu_launches=int(launches),
               launches_per_step=launches / total_steps, dtype="bf16" if w.net_kind == "conv" else "f32",
               config=dict(workload=w.name, n_agents=n, envs_per_agent=w.n_envs, n_steps=w.n_steps,
                           frames_per_step=frames_per_step, topology=topo_name, mode=mode_text,
                           l2="flushed between steps (252 MiB write)" if mode == "sync" else
                              "not flushed: a round's inputs and state (%.1f GB) exceed L2" % (rb / 1e9),
                           multi_gpu="replicas only" if world > 1 else "single"),
               roofline=roofline, round_roofline=round_roofline,
               wall_ms_per_step=1e3 * t_wall / total_steps,
               kernel_ms_per_step={k: round(v, 5) for k, v in sorted(per_class_ms.items(), key=lambda kv: -kv[1])})
    if is_async:
        rec["async"] = dict(mixes=mixes, skipped=skipped, mixed_fraction=mixed_frac,
                            staleness_mean=sum(b["staleness_sum"] - a["staleness_sum"] for a, b in zip(st0, st1)) / max(1, mixes),
                            staleness_max=max(b["staleness_max"] for b in st1))
        if group_sizes:
            rec["async"]["calls"] = len(group_sizes)
            rec["async"]["agents_per_call_mean"] = float(np.mean(group_sizes))
    if block_ms:
        rec["block_ms_per_step"] = [round(x, 4) for x in block_ms]

    # ------------------------------------------------------------------ end to end from host buffers
    if e2e:
        # pinned host -> device copy of every step's rollouts, the step, and a device -> host read of the step's
        # losses, all inside the timed region; copies run two steps ahead of the compute.  The asynchronous
        # workloads are driven without simulator delays here (the copies are the bound).
        h2d = sets[0].nbytes
        up_done = [torch.cuda.Event() for _ in range(n_sets)]

        def upload(j):
            sets[j].upload(up)
            up_done[j].record(up)

        def step_from_host(k):
            j = k % n_sets
            if mode == "sync":
                ext.wait_event(up_done[j])
                sync_step(sets[j])
            else:
                up_done[j].synchronize()       # the grouped calls run on streams of the library's own
                grouped_round(sets[j])

        esteps = max(K, int(math.ceil(MIN_REGION_S / max(est, h2d / 50e9))))
        for k in range(2):
            upload(k % n_sets)
            step_from_host(k)
            B.gala_losses_all(L.ctx, n)
        env.barrier()
        t0 = time.perf_counter()
        upload(0)
        if esteps > 1:
            upload(1 % n_sets)
        for k in range(esteps):
            step_from_host(k)
            if k + 2 < esteps:
                upload((k + 2) % n_sets)
            B.gala_losses_all(L.ctx, n)
        env.barrier()
        e2e_s = max_over_ranks(time.perf_counter() - t0)
        rec["e2e"] = dict(value=frames_per_step * esteps * world / e2e_s, unit=UNIT, h2d_bytes_per_step=int(h2d),
                          d2h_bytes_per_step=20 * n, steps=esteps)
    rec["_learner"] = (L, sets, ext)     # kept alive for legs that reuse the context; closed by the caller
    return rec


def close_record(env: Env, rec):
    L, sets, ext = rec.pop("_learner")
    del sets, ext
    import gc
    gc.collect()
    env.torch.cuda.synchronize()
    L.close()


def extras_c2(env: Env, rec, w: GI.Workload):
    """Pieces beyond the core step, on the 8-agent workload: distance from consensus, the synchronous A2C baseline
    (gradient all-reduce instead of gossip), Proposition 1's bound, the closed actor loop."""
    torch, B, LM = env.torch, env.B, env.LM
    L, sets, _ = rec["_learner"]
    n_sets = len(sets)
    t0 = time.perf_counter()
    reps = 20
    for _ in range(reps):
        dist = B.gala_consensus_distance(L.ctx)
    cons_ms = 1e3 * (time.perf_counter() - t0) / reps
    L2 = LM.Learner(w.n_agents, GI.COMPLETE, 0, w.net_kind, w.n_actions, w.n_envs, w.n_steps,
                    obs_dim=w.obs_dim, hidden=w.hidden)
    ext2 = torch.cuda.ExternalStream(B.gala_get_stream(L2.ctx, -1))
    for k in range(3):
        L2.step_sync(sets[k % n_sets])
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    L2.sync()
    e0.record(ext2)
    for k in range(20):
        L2.step_sync(sets[k % n_sets])
    e1.record(ext2)
    L2.sync()
    a2c_ms = e0.elapsed_time(e1) / 20
    L2.close()
    del ext2
    # Proposition 1 on this workload: identical initial parameters, eight synchronous rounds with the norm of
    # every round's step tracked; the measured distance from consensus beside the bound
    # b(k+1) = sigma_2(W_k) * (b(k) + ||alpha G(k)||), W_k the round's mixing matrix built from the library's
    # in-peers (equal weights over self and in-peers), sigma_2 its second singular value
    L3 = LM.Learner(w.n_agents, w.topo_kind, w.topo_peers, w.net_kind, w.n_actions, w.n_envs, w.n_steps,
                    obs_dim=w.obs_dim, hidden=w.hidden)
    B.gala_track_updates(L3.ctx, True)
    p1_dist, p1_bound, bnd = [], [], 0.0
    p1_W, p1_u, p1_prod = [], [], []
    for k in range(8):
        Wk = np.zeros((w.n_agents, w.n_agents))
        for i in range(w.n_agents):
            peers = [i] + B.gala_in_peers(L3.ctx, k, i)
            for j in peers:
                Wk[i, j] += 1.0 / len(peers)
        s2 = float(np.linalg.svd(Wk, compute_uv=False)[1]) if w.n_agents > 1 else 0.0
        L3.step_sync(sets[k % n_sets])
        p1_u.append(B.gala_update_norm(L3.ctx))
        bnd = s2 * (bnd + p1_u[-1])
        p1_dist.append(B.gala_consensus_distance(L3.ctx))
        p1_bound.append(bnd)
        # the same bound with the factor of every step taken from the product of the rounds since, as in the
        # proof: X(k+1) - mean = -sum_s (W_k ... W_s - 11^T/n) alpha G(s); for the exponential graphs a full
        # cycle of rounds averages exactly, which single-round factors cannot see
        p1_W.append(Wk)
        J = np.full_like(Wk, 1.0 / w.n_agents)
        P, tot = np.eye(w.n_agents), 0.0
        for s_ in range(k, -1, -1):
            P = P @ p1_W[s_]
            tot += float(np.linalg.norm(P - J, 2)) * p1_u[s_]
        p1_prod.append(tot)
    L3.close()
    # closed actor loop: every agent acts T times on the synthetic environment, learns and gossips, nothing
    # crosses the host; timed by the host clock between two synchronisations
    loop_iters = 10
    for i in range(w.n_agents):
        B.gala_actor_loop(L.ctx, i, 2, 12345)
    L.sync()
    t0 = time.perf_counter()
    for _ in range(loop_iters):
        for i in range(w.n_agents):
            B.gala_actor_loop(L.ctx, i, 1, 12345)
    L.sync()
    loop_s = time.perf_counter() - t0
    rec["closed_loop"] = dict(frames_per_s=w.frames_per_round * loop_iters / loop_s,
                              ms_per_round=1e3 * loop_s / loop_iters,
                              note="act x T + environment step x T + learn + gossip per agent on its own stream, "
                                   "synthetic on-GPU environment, host clock")
    # the same loop with all agents in lockstep: acting batched over the agents, then the synchronous round
    all_iters = 50
    B.gala_actor_loop_all(L.ctx, 4, 12345)
    L.sync()
    t0 = time.perf_counter()
    B.gala_actor_loop_all(L.ctx, all_iters, 12345)
    L.sync()
    all_s = time.perf_counter() - t0
    rec["closed_loop_lockstep"] = dict(frames_per_s=w.frames_per_round * all_iters / all_s,
                                       ms_per_round=1e3 * all_s / all_iters,
                                       note="T x (one forward pass of all agents, one draw + environment-step kernel "
                                            "of all agents) + the synchronous round, host clock")
    rec["extras"] = dict(consensus_distance=dist, consensus_call_ms=cons_ms,
                         consensus_bytes=int(w.n_agents * L.d * 4),
                         allreduce_a2c_ms_per_round=a2c_ms,
                         allreduce_a2c_frames_per_s=w.frames_per_round / (a2c_ms * 1e-3),
                         prop1=dict(distance=[round(x, 6) for x in p1_dist], bound=[round(x, 6) for x in p1_bound],
                                    bound_from_products=[round(x, 6) for x in p1_prod],
                                    holds=all(d_ <= min(b_, c_) * (1 + 1e-4)
                                              for d_, b_, c_ in zip(p1_dist, p1_bound, p1_prod))),
                         note="consensus_call_ms is a host-timed call (sync + one kernel + 8-byte read); "
                              "all-reduce rounds back to back without L2 flush")


def sweep_microbench(torch, B, pk):
    """Fused RMSProp + gossip pass alone on 32 agents x 1.7M fp32 parameters (and on the conv net's 1 693 875),
    100 rounds of the 1- and 2-peer exponential graphs.  All-agent form (gala_sweep_sync): 20 algorithmic bytes
    per parameter (read x, g, v; write x, v).  Per-agent form (gala_sweep_agents, all 32 agents in flight in one
    launch, every agent averaging): 24 + 4 p bytes (also the p in-peers' snapshots read, the own snapshot
    written)."""
    w = GI.WORKLOADS[3]
    n = w.n_agents
    hp = B.default_hparams(1, 1, max_grad_norm=0.0)
    st = torch.cuda.current_stream()
    out = {}

    def timed(fn, rounds=100):
        for k in range(5):
            fn(k)
        torch.cuda.synchronize()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(rounds)]
        for k in range(rounds):
            ev[k][0].record(st)
            fn(k)
            ev[k][1].record(st)
        torch.cuda.synchronize()
        ms = [a.elapsed_time(b) for a, b in ev]
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(st)
        for k in range(rounds):
            fn(k)
        e1.record(st)
        torch.cuda.synchronize()
        return median(ms), e0.elapsed_time(e1) / rounds

    for d in (w.sweep_only_d, 1_693_875):
        d_pad = (d + 3) // 4 * 4
        x, g, v = GI.sweep_state(n, d_pad, w.seed)
        tx, tg, tv = (torch.from_numpy(t).cuda() for t in (x, g, v))
        ts = torch.zeros((n, 3, d_pad), device="cuda")
        for s_ in range(3):
            ts[:, s_] = tx
        for peers in (1, 2):
            topo = B.gala_topology(B.GALA_TOPO_EXP, peers)
            med, b2b = timed(lambda k: B.gala_sweep_sync(tx, tg, tv, None, n, d_pad, topo, k, hp, st.cuda_stream))
            gbs = 20.0 * n * d_pad / (b2b * 1e-3) / 1e9
            out["sync_exp%d_d%d" % (peers, d)] = dict(
                form="all agents (gala_sweep_sync)", bytes_per_param=20, ms_per_round=b2b,
                ms_per_round_median_of_launches=med, achieved_gbs=gbs, frac_of_measured_peak=gbs / pk["hbm"],
                frac_of_8tbs=gbs / 8000.0)

            def agent_form(k, peers=peers):
                # round k of the exponential graph; version k was published into slot k % 3, version k + 1 goes to
                # slot (k + 1) % 3
                items = []
                for i in range(n):
                    plist = []
                    for j in range(peers):
                        off = 1 << ((peers * k + j) % 5)
                        plist.append(((i - off) % n, k % 3))
                    items.append((i, (k + 1) % 3, plist, True))
                B.gala_sweep_agents(tx, tg, tv, ts, None, n, 3, d_pad, items, hp, st.cuda_stream)

            med, b2b = timed(agent_form)
            bpp = 24 + 4 * peers
            gbs = float(bpp) * n * d_pad / (b2b * 1e-3) / 1e9
            out["agents_exp%d_d%d" % (peers, d)] = dict(
                form="per agent, 32 agents in one launch (gala_sweep_agents)", bytes_per_param=bpp, ms_per_round=b2b,
                ms_per_round_median_of_launches=med, achieved_gbs=gbs, frac_of_measured_peak=gbs / pk["hbm"],
                frac_of_8tbs=gbs / 8000.0)
        del tx, tg, tv, ts
    out["config"] = dict(workload=w.name, n_agents=n, d=[w.sweep_only_d, 1_693_875], rounds=100,
                         timing="ms_per_round: 100 launches back to back between two events; the median is over "
                                "per-launch event pairs",
                         l2="working set 653 MB (all-agent form) / 1.3 GB (per-agent form) > L2, no flush")
    return out


# which records a run produces: (key, workload index, mode)
FULL_SET = [("c5_async", 4, "async"), ("c5_async_noskew", 4, "async_noskew"), ("c5_sync", 4, "sync"),
            ("c5_sync_stragglers", 4, "sync_stragglers"), ("c3_sync", 2, "sync"), ("c2_sync", 1, "sync"),
            ("c1_sync", 0, "sync")]


def run_ours(args):
    env = Env(args)
    torch, B = env.torch, env.B
    clocks = ClockSampler(env.local)
    clocks.start()
    time.sleep(1.0)               # the sampler needs most of a second to deliver its first line
    if args.workload >= 0:
        mode = args.mode
        if mode == "auto":
            mode = "async" if args.workload == 4 else "sync"
        plan = [("head", args.workload, mode)]
    else:
        plan = FULL_SET
    records = {}
    for key, wi, mode in plan:
        w = GI.WORKLOADS[wi]
        rec = measure(env, w, mode, key, e2e=not args.no_e2e and mode != "sync_stragglers")
        if wi == 1 and mode == "sync" and env.rank == 0 and env.world == 1 and not args.no_extras:
            extras_c2(env, rec, w)
        close_record(env, rec)
        records[key] = rec
    head_key = plan[0][0]
    head = records[head_key]
    clocks.stop()
    for key, t0, t1 in env.spans:
        records[key]["clocks"] = clocks.window(t0, t1)
    line = dict(metric=METRIC, value=head["value"], unit=UNIT, n_gpus=env.world, steps=args.steps,
                warmup=max(3, args.warmup), ms_per_step=head["ms_per_step"], higher_is_better=True, scaling="weak",
                vs_baseline=None, dtype=head["dtype"], data="synthetic", config=head["config"],
                clocks=head["clocks"], e2e=head.get("e2e"), gpu_launches=head["gpu_launches"],
                roofline=head["roofline"], round_roofline=head["round_roofline"],
                timing=dict(ms_per_step="median over the timed steps", timed_steps=head["timed_steps"],
                            ms_per_step_mean=head["ms_per_step_mean"], min_region_s=MIN_REGION_S,
                            note="--steps K steps are repeated until the timed region lasts at least min_region_s"))
    for k in ("async", "wall_ms_per_step", "kernel_ms_per_step", "block_ms_per_step", "launches_per_step", "closed_loop",
              "closed_loop_lockstep", "extras"):
        if k in head:
            line[k] = head[k]
    if len(records) > 1:
        line["workloads"] = {k: v for k, v in records.items() if k != head_key}
        a, s = records.get("c5_async"), records.get("c5_sync_stragglers")
        if a and s:
            line["async_vs_sync_under_stragglers"] = dict(
                async_ms_per_round=a["ms_per_step"], sync_waiting_ms_per_round=s["ms_per_step"],
                speedup=s["ms_per_step"] / a["ms_per_step"],
                note="same simulator delay distribution; the synchronous loop starts a round when the slowest "
                     "agent's rollout has arrived (Sec. 5, computational performance)")
    if env.rank == 0 and env.world == 1 and not args.no_extras:
        line["sweep_microbench"] = sweep_microbench(torch, B, env.pk)
        if not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(GI.WORKLOADS[plan[0][1]])
    if env.rank == 0:
        print(json.dumps(line))
    if env.world > 1:
        env.dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=-1,
                    help="index into gala_inputs.WORKLOADS: only that workload (-1: all of them, the 64-agent "
                         "asynchronous one as the headline)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the end-to-end legs (host buffers, copies inside)")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the legs beyond the timed rounds and the end-to-end leg (consensus distance, all-reduce "
                         "baseline, closed actor loop, optimiser micro-benchmark, CPU oracle): for profiler runs")
    ap.add_argument("--mode", default="auto", choices=["auto", "sync", "async", "async_noskew", "sync_stragglers"],
                    help="with --workload; auto: asynchronous for workload 4, synchronous rounds otherwise")
    ap.add_argument("--lanes", type=int, default=0, help="streams the grouped calls alternate between (library default: 1)")
    ap.add_argument("--no-graphs", action="store_true", help="launch every kernel of a learner step directly (no graph replay)")
    ap.add_argument("--sweep-only", action="store_true",
                    help="run only the RMSProp + gossip micro-benchmark (32 agents x 1.7M parameters)")
    args = ap.parse_args()
    if args.sweep_only:
        import torch
        from paper_1906_04585_b200 import binding as B
        print(json.dumps(dict(metric="gossip-mix+RMSprop GB/s", sweep_microbench=sweep_microbench(torch, B, peaks()))))
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
