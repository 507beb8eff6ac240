#!/usr/bin/env python
"""Benchmark of the imitation-step hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A step is one pass of the whole path over all envs of the workload: policy
forward + Gaussian sampling on the current observations, then the fused env
step (reference lookup/FK, reward, flags, masked reset, next observation) on
that step's simulated body states.  Prints one JSON line (rank 0).

The timed region is a CUDA graph of K steps, replayed REPLAYS times; `value` is the median replay
(`replays` carries the spread), `sustained` a loop of replays at least a second long with the SM
clock sampled beside it.  With the default workload the other four configurations are measured too
(`other_configs`, each in a process of its own).

`--impl reference` times the CPU oracle on a bounded sample of the same
workload on the host cores (a deliberately plain program: a baseline, not a
target).

`--only env|policy|gae|ppo_loss|update` runs one piece in a plain timing loop and prints its own
JSON line: the entry point the kernel profiles under profiles/ were captured through.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2609_09821_b200 import workloads as W  # noqa: E402

DEFAULT_WORKLOAD = "cfg4_65536_smpl24"
METRIC = "env-steps/s (obs+reward+reset+policy fwd)"
UNIT = "env-steps/s"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


REPLAYS = 21            # replays of the K-step graph; the median is reported
SUSTAINED_SECONDS = 1.0

# dram__bytes_read.sum + dram__bytes_write.sum per launch from ncu captures of the kernels named in `capture`
# (one launch each, 65536 envs); None where the timed path runs another kernel variant than the captured one.
NCU_TRAFFIC = {
    "cfg4_65536_smpl24": dict(
        policy=dict(bytes=645075456, capture="linear_tc_hidden_pair_kernel<0, 0> x 3 + linear_tc_head_kernel<80>, one policy "
                                              "forward at 65536 envs (ncu --set full)"),
        env=dict(bytes=291532288, capture="env_step_kernel_small<0, 0, 0> writing fp32 and bf16 rows, one launch, "
                                          "65536 envs (ncu --set full)")),
}


def env_bytes_per_env(J: int) -> int:
    """Algorithmic HBM bytes of the env kernel per env-step: body states in, observation row,
    reward, flags out, per-env state read + written."""
    return 13 * J * 4 + (24 * J + 1) * 4 + 4 + 1 + 24


def mlp_flops_per_env(dims) -> int:
    return sum(2 * a * b for a, b in zip(dims[:-1], dims[1:]))


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx = gpu_index
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(self.idx), "--query-gpu=" + self.Q,
                                       "--format=csv,noheader,nounits", "-lms", "20"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self) -> dict:
        if self.p is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f:
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1])); mx.append(float(c[2])); power.append(float(c[3]))
            except ValueError:
                continue
            for name, v in zip(names, c[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        self.f.close()
        os.unlink(self.f.name)
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["no samples"])
        return dict(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), power_w_max=float(max(power)),
                    samples=len(sm), reasons=sorted(reasons))


# ----------------------------------------------------------------------------- CPU oracle leg
def oracle_leg(wl: W.Workload, skel, lib, pol, n_sample: int, steps: int, warmup: int, budget_s: float):
    """Times the oracle as it stands on `n_sample` envs of the workload; returns env-steps/s."""
    from oracle import oracle as O
    n = min(n_sample, wl.n_envs)
    osk = O.Skeleton(skel["parents"], skel["offsets"], skel["masses"])
    ocl = O.Clips(osk, lib["n_frames"], lib["fps"], lib["root_pos"], lib["local_quat"])
    cfg = O.make_env_config(wl.dt, wl.seed, W.REWARD_MULT, wl.h_min)
    cores = os.cpu_count() or 1
    env = O.Env(osk, ocl, cfg, n, n_threads=cores)
    state = dict(obs=env.reset_all(0), t=0.0, done=0)
    t_start = time.perf_counter()

    def consume(s, sim):
        sim = np.ascontiguousarray(sim.numpy())
        if state["t"] > budget_s and state["done"] >= 1:
            raise StopIteration
        t0 = time.perf_counter()
        O.policy_forward(pol["dims"], pol["W"], pol["b"], wl.sigma_action, wl.seed, s, state["obs"],
                         n_threads=cores)
        out = env.step(s, sim, want_terms=False)
        dt = time.perf_counter() - t0
        state["obs"] = out["obs"]
        if s > warmup:
            state["t"] += dt
            state["done"] += 1

    try:
        W.rollout_inputs(wl, skel, lib, lambda: (env.clip_id, env.t), consume, steps=warmup + steps)
    except StopIteration:
        pass
    done = max(state["done"], 1)
    return dict(value=n * done / max(state["t"], 1e-9), cores=cores, steps=done, n=n,
                ms_per_step=1e3 * state["t"] / done, wall_s=time.perf_counter() - t_start)


# ----------------------------------------------------------------------------- rollout-side pieces
# Timed on their own (not part of the metric).
def time_gae(B, wl, n, dev, stream, reps=20, T=None):
    """The advantage estimator over one rollout of T (default wl.steps) steps.  Its 17 B per env-step fit in L2, so a 256 MB
    buffer is read before every launch (reading leaves clean lines behind: a written buffer's write-back would
    be charged to the kernel)."""
    import torch
    T = T or wl.steps
    r_np, v_np, f_np = W.make_rollout_signals(T, n, wl.seed)
    r_d, v_d, f_d = (torch.from_numpy(a).to(dev) for a in (r_np, v_np, f_np))
    adv_d, ret_d = torch.empty((T, n), device=dev), torch.empty((T, n), device=dev)
    flush = torch.zeros(64 << 20, dtype=torch.int32, device=dev)
    t_gae = []
    for i in range(3 + reps):
        flush.sum()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        B.gae(r_d, v_d, f_d, adv_d, ret_d, 0.99, 0.95, True, stream=stream)
        b.record(stream)
        torch.cuda.synchronize()
        if i >= 3:
            t_gae.append(a.elapsed_time(b) * 1e-3)
    t_gae = float(np.median(t_gae))
    gae_bytes = T * n * 17 + n * 4
    return dict(T=T, seconds_per_launch=t_gae, algorithmic_bytes=gae_bytes, achieved_gbs=gae_bytes / t_gae / 1e9,
                l2="256 MB read before every launch")


def time_ppo_loss(B, wl, n, A, dev, stream, reps=20):
    """PPO minibatch loss: one of four minibatches of the rollout (T * n / 4 samples), moments + loss + finish."""
    import torch
    Mb = wl.steps * n // 4
    pb = {k: torch.from_numpy(v).to(dev) for k, v in W.make_ppo_batch(min(Mb, 65536), A, wl.seed, drift=0.02).items()}
    reps_rows = (Mb + pb["mean"].shape[0] - 1) // pb["mean"].shape[0]
    for k in ("mean", "action", "mean_old"):
        pb[k] = pb[k].repeat(reps_rows, 1)[:Mb].contiguous()
    for k in ("logp_old", "advantage", "value", "value_old", "returns"):
        pb[k] = pb[k].repeat(reps_rows)[:Mb].contiguous()
    ws, mom = B.ppo_workspace(), torch.empty(2, device=dev)
    outs = [torch.empty((Mb, A), device=dev), torch.empty(A, device=dev), torch.empty(Mb, device=dev),
            torch.empty(6, device=dev)]
    t_ppo = []
    for i in range(3 + reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        B.moments(pb["advantage"], mom, ws, stream=stream)
        B.ppo_loss(pb, *outs, ws, 0.2, 2.0, 2.5e-4, True, adv_moments=mom, stream=stream)
        b.record(stream)
        torch.cuda.synchronize()
        if i >= 3:
            t_ppo.append(a.elapsed_time(b) * 1e-3)
    t_ppo = float(np.median(t_ppo))
    ppo_bytes = Mb * ((3 * A + 5) * 4 + (A + 1) * 4 + 4)
    return dict(rows=Mb, A=A, seconds_per_launch=t_ppo, algorithmic_bytes=ppo_bytes, achieved_gbs=ppo_bytes / t_ppo / 1e9,
                l2="%.0f MB working set, larger than L2" % (ppo_bytes / 1e6))


def time_update(B, wl, pol, n, A, D, dev, stream, graph=True, reps=5):
    """One whole PPO minibatch update (actor + critic forward, loss, both backward passes, clip, Adam, learning
    rate) on 2 * n rows, a sixteenth of the rollout, through paper_2609_09821_b200.trainer."""
    import torch
    from paper_2609_09821_b200 import trainer as TR
    Mu = 2 * n
    adims, cdims_u = tuple(wl.mlp_dims), tuple(wl.mlp_dims[:-1]) + (1,)
    cwu = W.make_policy_weights(cdims_u, "bf16", wl.seed + 1)
    with torch.cuda.stream(stream):
        actor_t = TR.MlpTrainer(adims, pol["W"], pol["b"], Mu, stream=stream)
        critic_t = TR.MlpTrainer(cdims_u, cwu["W"], cwu["b"], Mu, stream=stream)
        upd = TR.PpoUpdater(actor_t, critic_t, torch.full((A,), -2.0), lr=5e-4, clip=0.2, value_coef=2.0)
        gen = torch.Generator(device=dev).manual_seed(wl.seed)
        for tr_ in (actor_t, critic_t):
            rows_ = tr_.input_rows(Mu)
            rows_.zero_()
            rows_[:, :D] = torch.randn((Mu, D), device=dev, generator=gen).to(torch.bfloat16)
        rnd = lambda *sh: torch.randn(*sh, device=dev, generator=gen)
        ub = dict(action=rnd(Mu, A) * 0.2, mean_old=rnd(Mu, A) * 0.2, log_std_old=torch.full((A,), -2.0, device=dev),
                  logp_old=rnd(Mu) + 60.0, advantage=rnd(Mu), value_old=rnd(Mu), returns=rnd(Mu))
        for i in range(2):
            upd.update(Mu, ub)
        stream.synchronize()
        up_graph = None
        if graph:
            # the update's ~100 launches are replayed from one CUDA graph, as a training loop would run them
            up_graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(up_graph, stream=stream):
                upd.update(Mu, ub)
        t_up = []
        for i in range(1 + reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            if up_graph is not None:
                up_graph.replay()
            else:
                upd.update(Mu, ub)
            b.record(stream)
            torch.cuda.synchronize()
            if i >= 1:
                t_up.append(a.elapsed_time(b) * 1e-3)
    t_up = float(np.median(t_up))
    up_flops = 3 * (mlp_flops_per_env(adims) + mlp_flops_per_env(cdims_u)) * Mu      # forward + two backward products
    return dict(rows=Mu, seconds_per_update=t_up, achieved_tflops=up_flops / t_up / 1e12,
                status=[actor_t.device_status(), critic_t.device_status()],
                launch="cuda_graph" if graph else "stream",
                note="forward + backward + Adam of actor and critic on one minibatch; flops = 3 x forward flops")


def time_gemm(B, shape, dev, stream, launches=20, reps=7):
    """C = relu(A W^T + b) in bf16 through im_gemm_bf16 for one (M, N, K): back-to-back launches, median of `reps`
    loops, and a comparison of the first 512 rows with a float32 product of the same operands."""
    import torch
    M, N, K = (int(x) for x in shape.split(","))
    gen = torch.Generator(device=dev).manual_seed(1)
    a = torch.randn((M, K), device=dev, generator=gen).to(torch.bfloat16)
    w = (torch.randn((N, K), device=dev, generator=gen) * K ** -0.5).to(torch.bfloat16)
    c = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
    bias = torch.zeros(N, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    for _ in range(3):
        B.gemm_bf16(a, w, c, bias, True, status, stream=stream)
    torch.cuda.synchronize()
    t = []
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(launches):
            B.gemm_bf16(a, w, c, bias, True, status, stream=stream)
        e1.record(stream)
        torch.cuda.synchronize()
        t.append(e0.elapsed_time(e1) / launches * 1e-3)
    sec = float(np.median(t))
    ref = torch.relu(a[:512].float() @ w.float().T)
    err = float((c[:512].float() - ref).abs().max() / (ref.abs().max() + 1e-9))
    return dict(M=M, N=N, K=K, seconds_per_launch=sec, achieved_tflops=2.0 * M * N * K / sec / 1e12,
                max_rel_err_first_512_rows=err, status=int(status.item()))


def only_rollout_piece(args):
    """`--only gae|ppo_loss|update|gemm`: that piece alone, in the loop the profiles of those kernels were taken from."""
    import torch
    from paper_2609_09821_b200 import binding as B
    B.load()
    wl = W.WORKLOADS[args.workload]
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    stream = torch.cuda.Stream()
    torch.cuda.set_stream(stream)
    n, A, D = args.envs or wl.n_envs, wl.act_dim, wl.obs_dim
    if args.only == "gae":
        res = time_gae(B, wl, n, dev, stream, reps=args.launches, T=args.horizon)
    elif args.only == "gemm":
        res = time_gemm(B, args.shape, dev, stream, launches=args.launches)
    elif args.only == "ppo_loss":
        res = time_ppo_loss(B, wl, n, A, dev, stream, reps=args.launches)
    else:
        pol = W.make_policy_weights(wl.mlp_dims, wl.mlp_dtype, wl.seed)
        res = time_update(B, wl, pol, n, A, D, dev, stream, graph=not args.no_graph, reps=args.launches)
    print(json.dumps(dict(only=args.only, workload=wl.name, **res)))


# ----------------------------------------------------------------------------- main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(W.WORKLOADS))
    ap.add_argument("--no-graph", action="store_true", help="plain stream launches instead of one CUDA graph")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-rollout-extras", action="store_true",
                    help="skip the separate timing of the value head and the advantage estimator")
    ap.add_argument("--no-other-configs", action="store_true",
                    help="skip the short device-resident runs of the other benchmark configurations")
    ap.add_argument("--replays", type=int, default=REPLAYS, help="replays of the K-step graph (median reported)")
    ap.add_argument("--only", default=None,
                    choices=["env", "policy", "gae", "ppo_loss", "update", "gemm", "fusion_probe"],
                    help="time one piece in a plain loop and print its own JSON line")
    ap.add_argument("--launches", type=int, default=40, help="launches of the --only loop")
    ap.add_argument("--envs", type=int, default=None, help="--only gae|ppo_loss|update: envs instead of the workload's")
    ap.add_argument("--horizon", type=int, default=None, help="--only gae: steps instead of the workload's")
    ap.add_argument("--shape", default="65536,1024,1024", help="--only gemm: M,N,K of the bf16 product")
    args = ap.parse_args()
    if args.only in ("gae", "ppo_loss", "update", "gemm"):
        return only_rollout_piece(args)

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    wl = W.WORKLOADS[args.workload]
    # default: eight rollouts of the workload's horizon, so that the timed region is long enough
    # (~0.1 s at the largest config) for clock samples to fall inside it
    K = args.steps if args.steps is not None else 8 * wl.steps
    Wm = max(args.warmup, 0)
    skel, lib, pol = W.build_scene(wl)
    J, D = skel["J"], wl.obs_dim
    config = dict(workload=wl.name, n_envs_per_gpu=wl.n_envs, bodies=J, obs_dim=D, mlp=list(wl.mlp_dims),
                  mlp_dtype=wl.mlp_dtype, clips=wl.n_clips, reward="multiplicative")

    if args.impl == "reference":
        if rank != 0:
            return
        res = oracle_leg(wl, skel, lib, pol, n_sample=2048, steps=K, warmup=Wm, budget_s=60.0)
        sample = "first %d envs of %s, %d steps" % (res["n"], wl.name, res["steps"])
        line = dict(metric=METRIC, value=res["value"], unit=UNIT, n_gpus=args.gpus, steps=res["steps"], warmup=Wm,
                    ms_per_step=res["ms_per_step"], higher_is_better=True, scaling="weak", vs_baseline=None,
                    dtype="f64", data="synthetic", impl="reference", config=config,
                    cpu_baseline=dict(value=res["value"], unit=UNIT, cores=res["cores"], kind="oracle", sample=sample),
                    e2e=dict(value=res["value"], unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
        print(json.dumps(line))
        return

    import torch
    from paper_2609_09821_b200 import binding as B
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    B.load()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    n = wl.n_envs                              # weak scaling: every rank runs the whole workload's env count
    env_base = rank * n
    ld = B.padded_ld(D)
    stream = torch.cuda.Stream()
    torch.cuda.set_stream(stream)

    g_skel = B.Skeleton(skel["parents"], skel["offsets"], skel["masses"])
    g_clips = B.Clips(g_skel, lib["n_frames"], lib["fps"], lib["root_pos"], lib["local_quat"])
    cfg = B.make_env_config(n, wl.dt, wl.seed, W.REWARD_MULT, wl.h_min, ld, env_id_base=env_base)
    env = B.Env(g_skel, g_clips, cfg, stream=stream)
    Wg = pol["W_bf16"] if pol["dtype"] == "bf16" else pol["W"]
    policy = B.Policy(pol["dims"], Wg, pol["b"], pol["dtype"], wl.sigma_action, wl.seed, n, env_id_base=env_base,
                      stream=stream)
    A = wl.act_dim
    staged = pol["dtype"] == "bf16"            # env writes bf16 rows straight into the policy's input buffer
    if staged:
        env.attach_policy(policy)

    def policy_forward(s):
        if staged:
            policy.forward_staged(s, n, mean, action)
        else:
            policy.forward(s, obs, mean, action)

    obs = env.new_obs()
    reward = torch.empty(n, device=dev)
    flags = torch.empty(n, dtype=torch.uint8, device=dev)
    mean = torch.empty((n, A), device=dev)
    action = torch.empty((n, A), device=dev)

    # ---- inputs: one pre-pass of the rollout fixes every env's (clip, time) per step; the simulator
    # ---- stand-in writes each step's body states straight into HBM
    total = Wm + K
    n_buf = min(total, 96)                     # bound device memory; longer runs cycle through the buffers
    env.reset_all(obs, 0)

    def get_state():
        c, t, _ = env.get_state()
        return c, t

    def consume(s, sim):
        policy_forward(s)
        env.step(s, sim, obs, reward, flags)

    sims = W.rollout_inputs(wl, skel, lib, get_state, consume, steps=n_buf, env_base=env_base, device=str(dev))
    torch.cuda.synchronize()
    if env.device_status() or policy.device_status():
        raise SystemExit("device status word set during the input pre-pass")

    def run_steps(first, count):
        for i in range(count):
            s = first + i
            policy_forward(s)
            env.step(s, sims[(s - 1) % n_buf], obs, reward, flags)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing
    env.reset_all(obs, 0)
    run_steps(1, Wm)
    torch.cuda.synchronize()
    graph = None
    launches_per_replay = None
    if not args.no_graph:
        c0, t0, l0 = env.get_state()
        obs0 = obs.clone()
        before = B.launch_count()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            run_steps(Wm + 1, K)
        launches_per_replay = B.launch_count() - before
        env.set_state(c0, t0, l0)
        obs.copy_(obs0)
        torch.cuda.synchronize()
    if args.only in ("env", "policy"):
        # plain loop over the step buffers (together larger than L2), the piece alone
        res = []
        for rep in range(3):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for i in range(args.launches):
                s_ = Wm + 1 + i
                if args.only == "env":
                    env.step(s_, sims[i % n_buf], obs, reward, flags)
                else:
                    policy_forward(s_)
            b.record(stream)
            torch.cuda.synchronize()
            res.append(a.elapsed_time(b) / args.launches * 1e3)
        if rank == 0:
            print(json.dumps(dict(only=args.only, workload=wl.name, us_per_launch=res, launches=args.launches,
                                  bf16_rows=bool(staged), reset_fraction=float((flags != 0).float().mean()))))
        return

    if args.only == "fusion_probe":
        # What fusing the env step with the policy's first layer could save in memory traffic: (a) the env step with
        # and without the bf16 rows it leaves for the policy; (b) the policy forward on rows that are still in L2
        # (the same launch repeated) against rows that have to come from HBM (256 MB read in between).
        def loop(fn, n_l=args.launches, between=None):
            out = []
            for rep in range(3):
                tot = 0.0
                for i in range(n_l):
                    if between is not None:
                        between()
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a.record(stream)
                    fn(i)
                    b.record(stream)
                    torch.cuda.synchronize()
                    tot += a.elapsed_time(b)
                out.append(tot / n_l * 1e3)
            return float(np.median(out))
        res = dict(only="fusion_probe", workload=wl.name)
        res["env_fp32_and_bf16_rows_us"] = loop(lambda i: env.step(Wm + 1 + i, sims[i % n_buf], obs, reward, flags))
        if staged:
            env.attach_policy(None)
            res["env_fp32_rows_only_us"] = loop(lambda i: env.step(Wm + 1 + i, sims[i % n_buf], obs, reward, flags))
            env.attach_policy(policy)
            env.step(Wm + 1, sims[0], obs, reward, flags)
        flush = torch.zeros(64 << 20, dtype=torch.int32, device=dev)
        res["policy_rows_in_l2_us"] = loop(lambda i: policy_forward(Wm + 1 + i))
        res["policy_rows_from_hbm_us"] = loop(lambda i: policy_forward(Wm + 1 + i), between=lambda: flush.sum())
        if rank == 0:
            print(json.dumps(res))
        return

    sampler = ClockSampler(local_rank)
    reps = max(1, args.replays) if graph is not None else 1
    evs_r = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
    barrier()
    sampler.start()
    before = B.launch_count()
    for ev0, ev1 in evs_r:
        ev0.record(stream)
        if graph is not None:
            graph.replay()
        else:
            run_steps(Wm + 1, K)
        ev1.record(stream)
    barrier()
    clocks = sampler.stop()
    launches = launches_per_replay if graph is not None else B.launch_count() - before
    times = np.array([a.elapsed_time(b) for a, b in evs_r])
    if world > 1:
        tmax = torch.from_numpy(times).to(dev)
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)        # every replay takes as long as its slowest rank
        times = tmax.cpu().numpy()
    ms = float(np.median(times))
    replays = dict(count=int(reps), ms_median=ms, ms_min=float(times.min()), ms_max=float(times.max()),
                   note="each replay is the K-step graph; value = n_envs * K / median")

    # ---- the same graph replayed back to back for at least a second: the settled figure under the power cap
    sustained = None
    if graph is not None and SUSTAINED_SECONDS > 0:
        n_rep = max(int(np.ceil(SUSTAINED_SECONDS * 1e3 / ms)), 2)
        s_sampler = ClockSampler(local_rank)
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        s_sampler.start()
        ev0.record(stream)
        for _ in range(n_rep):
            graph.replay()
        ev1.record(stream)
        barrier()
        s_clocks = s_sampler.stop()
        s_ms = ev0.elapsed_time(ev1)
        if world > 1:
            tmax = torch.tensor([s_ms], device=dev)
            dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
            s_ms = float(tmax.item())
        sustained = dict(value=world * n * K * n_rep / (s_ms * 1e-3), unit=UNIT, seconds=s_ms * 1e-3, replays=n_rep,
                         ms_per_step=s_ms / (K * n_rep), clocks=s_clocks,
                         ms_per_step_times_sm_mhz=(s_ms / (K * n_rep)) * s_clocks["sm_mhz"] if s_clocks.get("sm_mhz") else None)

    # ---- per-call breakdown (stream launches with events around each call) for the rooflines
    env.reset_all(obs, 0)
    run_steps(1, Wm)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K)]
    torch.cuda.synchronize()
    for i in range(K):
        s = Wm + 1 + i
        evs[i][0].record(stream)
        policy_forward(s)
        evs[i][1].record(stream)
        env.step(s, sims[(s - 1) % n_buf], obs, reward, flags)
        evs[i][2].record(stream)
    torch.cuda.synchronize()
    t_pol = float(np.mean([e[0].elapsed_time(e[1]) for e in evs])) * 1e-3
    t_env = float(np.mean([e[1].elapsed_time(e[2]) for e in evs])) * 1e-3

    # ---- rollout-side calls, timed on their own (not part of the metric): critic forward on the rows the
    # ---- env staged for the actor, and the advantage estimator over one rollout of wl.steps steps.  The
    # ---- estimator's 17 B per env-step fit in L2, so a 256 MB buffer is read before every launch (reading
    # ---- leaves clean lines behind: a written buffer's write-back would be charged to the kernel).
    extras = None
    if not args.no_rollout_extras and rank == 0:
        reps = 20
        extras = dict(gae=time_gae(B, wl, n, dev, stream, reps), ppo_loss=time_ppo_loss(B, wl, n, A, dev, stream, reps))
        if staged:
            extras["ppo_update"] = time_update(B, wl, pol, n, A, D, dev, stream)
        if staged:
            cdims = tuple(wl.mlp_dims[:-1]) + (1,)
            cw = W.make_policy_weights(cdims, "bf16", wl.seed + 1)
            critic = B.Policy(cdims, cw["W_bf16"], cw["b"], "bf16", 1.0, wl.seed, n, stream=stream)
            value = torch.empty((n, 1), device=dev)
            t_v = []
            for i in range(3 + reps):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                critic.value_forward_staged(n, value, src=policy)
                b.record(stream)
                torch.cuda.synchronize()
                if i >= 3:
                    t_v.append(a.elapsed_time(b) * 1e-3)
            t_v = float(np.median(t_v))
            cflops = mlp_flops_per_env(cdims) * n
            extras["value_head"] = dict(dims=list(cdims), seconds_per_launch=t_v, achieved_tflops=cflops / t_v / 1e12)
            del critic
            # policy serving: the env step asked for the policy's bf16 rows only (no fp32 observation output);
            # back-to-back launches over the step buffers, which together exceed L2
            t_s = []
            for i in range(3 + reps):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                for j in range(8):
                    env.step(Wm + K + 1 + 8 * i + j, sims[(8 * i + j) % n_buf], None, reward, flags)
                b.record(stream)
                torch.cuda.synchronize()
                if i >= 3:
                    t_s.append(a.elapsed_time(b) * 1e-3 / 8)
            extras["env_step_bf16_rows_only"] = dict(seconds_per_launch=float(np.median(t_s)),
                                                     note="im_env_step with obs_out == NULL while attached to the policy")

    # ---- end to end through the host-buffer entry point: pinned host inputs, results read back
    e2e = None
    if not args.no_e2e:
        n_host = min(n_buf, 16)                    # bound pinned memory; the host buffers are cycled
        host_sims = [s.cpu().pin_memory() for s in sims[:n_host]]
        act_h = torch.empty((n, A)).pin_memory()
        rew_h = torch.empty(n).pin_memory()
        fl_h = torch.empty(n, dtype=torch.uint8).pin_memory()
        env.reset_all_host(0)
        for s in range(1, Wm + 1):
            B.step_host(env, policy, s, host_sims[(s - 1) % n_host], act_h, rew_h, fl_h)
        barrier()
        t0 = time.perf_counter()
        for s in range(Wm + 1, Wm + K + 1):
            B.step_host(env, policy, s, host_sims[(s - 1) % n_host], act_h, rew_h, fl_h)
        torch.cuda.synchronize()
        e2e_s = time.perf_counter() - t0
        if world > 1:
            tmax = torch.tensor([e2e_s], device=dev)
            dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
            e2e_s = float(tmax.item())
        e2e = dict(value=world * n * K / e2e_s, unit=UNIT, h2d_bytes_per_step=13 * J * n * 4,
                   d2h_bytes_per_step=n * (A * 4 + 4 + 1), ms_per_step=1e3 * e2e_s / K,
                   timer="host clock around K calls that each wait for the stream")
        del host_sims

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    flops = mlp_flops_per_env(wl.mlp_dims) * n
    env_bytes = env_bytes_per_env(J) * n
    tf = flops / t_pol / 1e12
    gbs = env_bytes / t_env / 1e9
    tensor_peak = peaks["bf16_tflops_sustained"]
    traffic = NCU_TRAFFIC.get(wl.name, dict(policy=dict(bytes=None, capture=None), env=dict(bytes=None, capture=None)))
    # the K-step replays last milliseconds: the burst peak is the denominator that applies to them; the
    # fraction of the sustained peak is given beside it (it applies to the `sustained` loop)
    roofline = dict(bound="tensor", kernel="policy forward (GEMM chain + Gaussian head)", achieved=tf,
                    peak=peaks["bf16_tflops"], unit="TFLOP/s", frac=tf / peaks["bf16_tflops"],
                    frac_burst=tf / peaks["bf16_tflops"], frac_sustained=tf / tensor_peak,
                    peak_sustained=tensor_peak, traffic=traffic["policy"]["bytes"], traffic_capture=traffic["policy"]["capture"],
                    peak_source="%s bf16 burst (timed region of milliseconds)" % peaks["source"], seconds_per_launch=t_pol)
    roofline_env = dict(bound="hbm", kernel="env_step_kernel", achieved=gbs, peak=peaks["hbm_gbs"], unit="GB/s",
                        frac=gbs / peaks["hbm_gbs"], traffic=traffic["env"]["bytes"], traffic_capture=traffic["env"]["capture"],
                        peak_source="%s copy" % peaks["source"],
                        seconds_per_launch=t_env, algorithmic_bytes=env_bytes)
    if wl.mlp_dtype != "bf16":
        roofline["bound"] = "alu"
        roofline["peak_source"] = "fp32 SIMT path: tensor peak shown for scale only"
    config.update(launch="cuda_graph" if graph is not None else "stream",
                  l2="every step reads its own %.0f MB body-state buffer and rewrites the %.0f MB observation "
                     "buffer (%d distinct step buffers)" % (13 * J * n * 4 / 1e6, n * ld * 4 / 1e6, n_buf),
                  ld_obs=ld, parallelism="envs sharded across GPUs, no collective" if world > 1 else "single GPU")
    line = dict(metric=METRIC, value=world * n * K / (ms * 1e-3), unit=UNIT, n_gpus=world, steps=K, warmup=Wm,
                ms_per_step=ms / K, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="bf16" if wl.mlp_dtype == "bf16" else "f32", data="synthetic", config=config,
                clocks=clocks, gpu_launches=int(launches), roofline=roofline, roofline_env=roofline_env,
                breakdown_ms=dict(policy_forward=t_pol * 1e3, env_step=t_env * 1e3), replays=replays)
    if sustained is not None:
        line["sustained"] = sustained
    if e2e is not None:
        line["e2e"] = e2e
    if extras is not None:
        extras["gae"]["frac_of_hbm_peak"] = extras["gae"]["achieved_gbs"] / peaks["hbm_gbs"]
        extras["ppo_loss"]["frac_of_hbm_peak"] = extras["ppo_loss"]["achieved_gbs"] / peaks["hbm_gbs"]
        if "ppo_update" in extras:
            extras["ppo_update"]["frac_of_tensor_peak"] = extras["ppo_update"]["achieved_tflops"] / tensor_peak
        if "value_head" in extras:
            extras["value_head"]["frac_of_tensor_peak"] = extras["value_head"]["achieved_tflops"] / tensor_peak
        line["rollout_extras"] = extras
    if world == 1 and not args.no_other_configs and args.workload == DEFAULT_WORKLOAD:
        # the other configurations, device-resident numbers only, each in a process of its own (this one's
        # buffers are released first); the headline stays the default workload's
        import subprocess
        import sys
        del graph
        torch.cuda.empty_cache()
        others = {}
        for name in sorted(W.WORKLOADS):
            if name == wl.name:
                continue
            cmd = [sys.executable, os.path.abspath(__file__), "--workload", name, "--warmup", str(max(Wm, 3)),
                   "--no-cpu-baseline", "--no-e2e", "--no-rollout-extras", "--no-other-configs"]
            try:
                out = subprocess.run(cmd, capture_output=True, text=True, timeout=180)
                d = json.loads(out.stdout.strip().splitlines()[-1])
                others[name] = dict(value=d["value"], unit=UNIT, ms_per_step=d["ms_per_step"], steps=d["steps"],
                                    n_envs=d["config"]["n_envs_per_gpu"], dtype=d["dtype"], replays=d["replays"],
                                    sustained=d.get("sustained", {}).get("value"),
                                    roofline=d["roofline"] if d["dtype"] == "bf16" else None,
                                    roofline_env=d["roofline_env"], breakdown_ms=d["breakdown_ms"],
                                    sm_mhz=d["clocks"].get("sm_mhz"))
            except Exception as exc:                     # a side measurement must not take the headline down with it
                others[name] = dict(error=repr(exc)[:200])
        line["other_configs"] = others
    if not args.no_cpu_baseline:
        res = oracle_leg(wl, skel, lib, pol, n_sample=2048, steps=64, warmup=1, budget_s=15.0)
        line["cpu_baseline"] = dict(value=res["value"], unit=UNIT, cores=res["cores"], kind="oracle",
                                    sample="first %d envs of %s, %d steps" % (res["n"], wl.name, res["steps"]))
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
