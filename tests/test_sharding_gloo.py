"""Host-side logic of the multi-GPU path with two gloo ranks on CPU: envs are split in contiguous
blocks, each rank runs its shard with global env ids, nothing is exchanged on the data path, and
the gathered result equals the unsplit run.  The benchmark's timing reduction (max over ranks) is
exercised the same way."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import oracle as O
from paper_2609_09821_b200 import workloads as W

N_TOTAL = 101          # not divisible by the world size


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _run_shard(first, count, steps):
    wl = W.WORKLOADS["cfg5_reset_heavy"]
    skel, lib, pol = W.build_scene(wl)
    osk = O.Skeleton(skel["parents"], skel["offsets"], skel["masses"])
    ocl = O.Clips(osk, lib["n_frames"], lib["fps"], lib["root_pos"], lib["local_quat"])
    cfg = O.make_env_config(wl.dt, wl.seed, W.REWARD_MULT, wl.h_min)
    ids = np.arange(first, first + count, dtype=np.uint32)
    env = O.Env(osk, ocl, cfg, count, ids, n_threads=1)
    env.reset_all(0)
    # the simulated states of the unsplit batch, cut to this shard: every rank can regenerate them
    full = O.Env(osk, ocl, cfg, N_TOTAL, n_threads=1)
    full.reset_all(0)
    flags, obs = [], []
    for s in range(1, steps + 1):
        sim = W.synth_sim_state(skel, lib, full.clip_id, full.t.astype(np.float64) + wl.dt, s, wl)
        full.step(s, sim.copy(), want_terms=False)
        out = env.step(s, np.ascontiguousarray(sim[:, first:first + count]), want_terms=False)
        flags.append(out["flags"])
        obs.append(out["obs"])
    return np.stack(flags), np.stack(obs), env.clip_id.copy(), env.t.copy()


def _worker(rank, world, port, steps, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    first, count = W.shard_envs(N_TOTAL, world, rank)
    flags, obs, clip, t = _run_shard(first, count, steps)
    # pad to the largest shard so that all_gather sees equal shapes
    cmax = (N_TOTAL + world - 1) // world
    pack = torch.zeros((steps, cmax, obs.shape[2] + 3), dtype=torch.float64)
    pack[:, :count, :obs.shape[2]] = torch.from_numpy(obs)
    pack[:, :count, -3] = torch.from_numpy(flags.astype(np.float64))
    pack[:, :count, -2] = torch.from_numpy(clip.astype(np.float64))
    pack[:, :count, -1] = torch.from_numpy(t.astype(np.float64))
    gathered = [torch.zeros_like(pack) for _ in range(world)]
    dist.all_gather(gathered, pack)
    # the benchmark's timing rule: every rank reports the slowest rank's time
    tmax = torch.tensor([10.0 + rank])
    dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
    if rank == 0:
        parts = []
        for r in range(world):
            f, c = W.shard_envs(N_TOTAL, world, r)
            parts.append(gathered[r][:, :c])
        q.put((torch.cat(parts, dim=1).numpy(), float(tmax.item())))
    dist.barrier()
    dist.destroy_process_group()


def test_shard_partition_covers_everything():
    for n, w in [(101, 2), (65536, 8), (7, 8), (64, 1)]:
        spans = [W.shard_envs(n, w, r) for r in range(w)]
        assert spans[0][0] == 0 and sum(c for _, c in spans) == n
        for (f0, c0), (f1, _) in zip(spans, spans[1:]):
            assert f0 + c0 == f1
        assert max(c for _, c in spans) - min(c for _, c in spans) <= 1


def test_two_ranks_reproduce_the_unsplit_rollout():
    steps, world = 4, 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, steps, q)) for r in range(world)]
    for p in procs:
        p.start()
    merged, tmax = q.get(timeout=240)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    flags, obs, clip, t = _run_shard(0, N_TOTAL, steps)
    np.testing.assert_array_equal(merged[:, :, :-3], obs)
    np.testing.assert_array_equal(merged[:, :, -3], flags.astype(np.float64))
    np.testing.assert_array_equal(merged[-1, :, -2], clip.astype(np.float64))
    np.testing.assert_array_equal(merged[-1, :, -1], t.astype(np.float64))
    assert (flags != 0).any()                      # resets happened, so the Philox counters mattered
    assert tmax == 11.0
