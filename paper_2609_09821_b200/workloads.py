"""Seeded synthetic inputs for the imitation-step hot path.

This module is the only code shared by the CUDA path's callers and the CPU
oracle's callers.  It produces *inputs* only: skeletons, motion-clip
libraries, a stand-in for the physics simulator's body states, and policy
weights.  It evaluates none of the method's steps (no keyframe lookup, no
slerp, no reward, no reset rule, no observation, no MLP); the simulator
stand-in evaluates the *analytic* motion the keyframes were sampled from and
runs its own vectorised numpy kinematics, the way a physics engine would own
its kinematics.  Random numbers come from numpy's seeded bit generators; the
Philox streams the method itself draws (reset, action noise) are implemented
separately inside the CUDA library and inside the oracle.

The paper trains on five captured motions and an AMASS split (Section 6.1);
those are not available offline, so smooth seeded clips with the same
structure (30 Hz keyframes of root position + per-joint local quaternions,
w,x,y,z) stand in for them.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Callable, Dict, List, Optional, Sequence, Tuple

import numpy as np

# ----------------------------------------------------------------------------
# Skeleton topologies named by the benchmark configurations.
# ----------------------------------------------------------------------------
PARENTS_15 = [-1, 0, 1, 2, 1, 4, 5, 1, 7, 8, 0, 10, 11, 0, 13]
PARENTS_24 = [-1, 0, 0, 0, 1, 2, 3, 4, 5, 6, 7, 8, 9, 9, 9, 12, 13, 14, 16, 17,
              18, 19, 20, 21]

REWARD_TERMS = ("pose", "vel", "ee_pos", "ee_rot", "com", "body_pos", "body_vel")

# Reward presets.  MULT is the multiplicative form of Section 6.1; the weights
# the paper prints (pose 12, COM 8, end-effector rotation 1) are Table 4's
# "Selected" column, the two it never prints (velocity, end-effector position)
# are user parameters set here to 0.1 and 40.  FIG5 is the additive special
# case printed in Figure 5.
REWARD_MULT = dict(mode=0, a=[0.0] * 7, w=[12.0, 0.1, 40.0, 1.0, 8.0, 0.0, 0.0])
REWARD_FIG5 = dict(mode=1, a=[0.0, 0.0, 0.0, 0.0, 0.15, 0.60, 0.25],
                   w=[0.0, 0.0, 0.0, 0.0, 8.0, 4.0, 0.25])
REWARD_ADD4 = dict(mode=1, a=[0.65, 0.1, 0.15, 0.0, 0.1, 0.0, 0.0],
                   w=[2.0, 0.1, 40.0, 0.0, 10.0, 0.0, 0.0])


@dataclasses.dataclass(frozen=True)
class Workload:
    """One benchmark configuration (shapes and noise model only)."""
    name: str
    n_envs: int
    skeleton: str            # "humanoid15" | "smpl24"
    n_clips: int
    frames: Tuple[int, int]  # (lo, hi) inclusive keyframe-count range
    steps: int
    mlp_dims: Tuple[int, ...]
    mlp_dtype: str           # "f32" | "bf16"
    sigma_q: float = 0.05    # joint-rotation noise, rad
    sigma_root: float = 0.02 # root position noise, m
    sigma_vel: float = 0.1   # velocity noise
    h_min: float = 0.3       # early-termination root height, m
    fps: float = 30.0
    dt: float = 1.0 / 30.0
    sigma_action: float = 0.1
    seed: int = 0

    @property
    def n_bodies(self) -> int:
        return 15 if self.skeleton == "humanoid15" else 24

    @property
    def obs_dim(self) -> int:
        return 24 * self.n_bodies + 1

    @property
    def act_dim(self) -> int:
        return self.mlp_dims[-1]


WORKLOADS: Dict[str, Workload] = {
    w.name: w for w in [
        Workload("cfg1_tiny64", 64, "humanoid15", 1, (60, 60), 10,
                 (361, 1024, 512, 28), "f32"),
        Workload("cfg2_4096", 4096, "humanoid15", 1, (150, 150), 32,
                 (361, 1024, 512, 28), "bf16"),
        Workload("cfg3_16384_lib32", 16384, "humanoid15", 32, (60, 600), 32,
                 (361, 1024, 512, 28), "bf16"),
        Workload("cfg4_65536_smpl24", 65536, "smpl24", 32, (60, 600), 32,
                 (577, 1024, 1024, 512, 69), "bf16"),
        Workload("cfg5_reset_heavy", 16384, "humanoid15", 32, (60, 600), 64,
                 (361, 2048, 1024, 28), "bf16", sigma_q=0.3, h_min=0.8),
    ]
}


def _rng(seed: int, *stream: int) -> np.random.Generator:
    """Independent seeded stream; `stream` words separate uses and steps."""
    return np.random.Generator(np.random.Philox(
        np.random.SeedSequence([int(seed) & 0xFFFFFFFF, *[int(s) & 0xFFFFFFFF for s in stream]])))


# ----------------------------------------------------------------------------
# Skeleton
# ----------------------------------------------------------------------------
def make_skeleton(kind: str, seed: int = 0) -> dict:
    """Bone offsets = seeded unit directions x U[0.05, 0.45] m; masses U[1, 10] kg."""
    parents = np.asarray(PARENTS_15 if kind == "humanoid15" else PARENTS_24, np.int32)
    J = parents.shape[0]
    g = _rng(seed, 16)
    d = g.standard_normal((J, 3))
    d /= np.linalg.norm(d, axis=1, keepdims=True)
    length = g.uniform(0.05, 0.45, size=(J, 1))
    offsets = (d * length).astype(np.float32)
    offsets[0] = 0.0
    masses = g.uniform(1.0, 10.0, size=J).astype(np.float32)
    has_child = np.zeros(J, bool)
    has_child[parents[1:]] = True
    ee = np.nonzero(~has_child)[0].astype(np.int32)
    return dict(kind=kind, J=J, parents=parents, offsets=offsets, masses=masses, ee_ids=ee)


# ----------------------------------------------------------------------------
# Quaternion helpers for the generators (w,x,y,z; Hamilton; float64 arrays).
# ----------------------------------------------------------------------------
def _qmul(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    aw, ax, ay, az = np.moveaxis(a, -1, 0)
    bw, bx, by, bz = np.moveaxis(b, -1, 0)
    return np.stack([aw * bw - ax * bx - ay * by - az * bz,
                     aw * bx + ax * bw + ay * bz - az * by,
                     aw * by - ax * bz + ay * bw + az * bx,
                     aw * bz + ax * by - ay * bx + az * bw], axis=-1)


def _qconj(a: np.ndarray) -> np.ndarray:
    return a * np.array([1.0, -1.0, -1.0, -1.0])


def _qrot(q: np.ndarray, v: np.ndarray) -> np.ndarray:
    w = q[..., :1]
    u = q[..., 1:]
    t = 2.0 * np.cross(u, v)
    return v + w * t + np.cross(u, t)


def _qexp_half(r: np.ndarray) -> np.ndarray:
    """Unit quaternion of the rotation vector r (angle = |r|)."""
    ang = np.linalg.norm(r, axis=-1, keepdims=True)
    half = 0.5 * ang
    k = np.where(ang > 1e-12, np.sin(half) / np.maximum(ang, 1e-300), 0.5)
    return np.concatenate([np.cos(half), k * r], axis=-1)


def _qlog_rotvec(q: np.ndarray) -> np.ndarray:
    """Rotation vector (shortest arc) of a unit quaternion."""
    q = np.where(q[..., :1] < 0, -q, q)
    n = np.linalg.norm(q[..., 1:], axis=-1, keepdims=True)
    ang = 2.0 * np.arctan2(n, q[..., :1])
    k = np.where(n > 1e-12, ang / np.maximum(n, 1e-300), 2.0)
    return k * q[..., 1:]


# ----------------------------------------------------------------------------
# Motion clips: r_j(tau) = sum_m A_jm sin(2 pi 0.5 m tau + phi_jm), q = exp(r/2)
# root path (1 m/s * tau, 0, ROOT_HEIGHT + 0.05 sin 2 pi tau).  ROOT_HEIGHT = 0.82 m puts the
# per-step reset rate of the reset-heavy workload (h_min = 0.8 m) at 11-34 %, mean 16 %.
# ----------------------------------------------------------------------------
N_HARM = 3
ROOT_HEIGHT = 0.82


def make_clip_library(J: int, n_clips: int, frames: Tuple[int, int], fps: float = 30.0,
                      seed: int = 0) -> dict:
    g = _rng(seed, 17)
    lo, hi = frames
    n_frames = g.integers(lo, hi + 1, size=n_clips).astype(np.int32)
    amp = g.uniform(-0.5, 0.5, size=(n_clips, J, N_HARM, 3))
    phi = g.uniform(0.0, 2.0 * math.pi, size=(n_clips, J, N_HARM, 3))
    lib = dict(J=J, C=n_clips, n_frames=n_frames,
               fps=np.full(n_clips, fps, np.float32), amp=amp, phi=phi)
    roots, quats = [], []
    for c in range(n_clips):
        tau = np.arange(int(n_frames[c]), dtype=np.float64) / fps
        p, q = analytic_pose(lib, np.full(tau.shape, c, np.int64), tau)
        roots.append(p)
        quats.append(q)
    lib["root_pos"] = np.concatenate(roots).astype(np.float32)
    lib["local_quat"] = np.concatenate(quats).astype(np.float32)
    lib["frame_start"] = np.concatenate([[0], np.cumsum(n_frames)[:-1]]).astype(np.int64)
    return lib


def analytic_pose(lib: dict, clip_id: np.ndarray, tau: np.ndarray):
    """Root position [n,3] and local joint quaternions [n,J,4] of the analytic motion."""
    amp = lib["amp"][clip_id]            # [n,J,H,3]
    phi = lib["phi"][clip_id]
    m = np.arange(1, N_HARM + 1, dtype=np.float64).reshape(1, 1, N_HARM, 1)
    arg = 2.0 * math.pi * 0.5 * m * tau.reshape(-1, 1, 1, 1) + phi
    r = (amp * np.sin(arg)).sum(axis=2)  # [n,J,3]
    q = _qexp_half(r)
    p = np.stack([1.0 * tau, np.zeros_like(tau), ROOT_HEIGHT + 0.05 * np.sin(2.0 * math.pi * tau)], axis=-1)
    return p, q


def _kinematics(skel: dict, root_p: np.ndarray, q_l: np.ndarray):
    """World positions [n,J,3] and rotations [n,J,4] of every body (numpy, small inputs)."""
    J = skel["J"]
    par = skel["parents"]
    off = skel["offsets"].astype(np.float64)
    p = np.empty(q_l.shape[:-1] + (3,))
    q = np.empty_like(q_l)
    p[:, 0] = root_p
    q[:, 0] = q_l[:, 0]
    for j in range(1, J):
        a = int(par[j])
        q[:, j] = _qmul(q[:, a], q_l[:, j])
        p[:, j] = p[:, a] + _qrot(q[:, a], np.broadcast_to(off[j], p[:, a].shape))
    return p, q


# ---- the simulator stand-in proper, in torch so that it runs on whichever device holds the
# ---- rollout (a few million env-steps per benchmark run would take minutes in numpy)
def _t_qmul(a, b):
    import torch
    aw, ax, ay, az = a.unbind(-1)
    bw, bx, by, bz = b.unbind(-1)
    return torch.stack([aw * bw - ax * bx - ay * by - az * bz,
                        aw * bx + ax * bw + ay * bz - az * by,
                        aw * by - ax * bz + ay * bw + az * bx,
                        aw * bz + ax * by - ay * bx + az * bw], dim=-1)


def _t_qrot(q, v):
    import torch
    w, u = q[..., :1], q[..., 1:]
    t = 2.0 * torch.linalg.cross(u, v)
    return v + w * t + torch.linalg.cross(u, t)


def _t_qexp_half(r):
    import torch
    ang = torch.linalg.norm(r, dim=-1, keepdim=True)
    half = 0.5 * ang
    k = torch.where(ang > 1e-12, torch.sin(half) / ang.clamp_min(1e-300), torch.full_like(ang, 0.5))
    return torch.cat([torch.cos(half), k * r], dim=-1)


def _t_qlog_rotvec(q):
    import torch
    q = torch.where(q[..., :1] < 0, -q, q)
    n = torch.linalg.norm(q[..., 1:], dim=-1, keepdim=True)
    ang = 2.0 * torch.atan2(n, q[..., :1])
    k = torch.where(n > 1e-12, ang / n.clamp_min(1e-300), torch.full_like(n, 2.0))
    return k * q[..., 1:]


def _motion_coeffs(lib: dict, device):
    """[C, J, 2H, 3] table so that r = coeffs . [sin(w_m tau), cos(w_m tau)] (angle addition)."""
    import torch
    key = "_coef_%s" % (device,)
    if key not in lib:
        amp, phi = lib["amp"], lib["phi"]                      # [C,J,H,3]
        coef = np.concatenate([amp * np.cos(phi), amp * np.sin(phi)], axis=2)
        lib[key] = torch.from_numpy(coef).to(device)
    return lib[key]


def _t_analytic_pose(lib: dict, clip_id, tau):
    import torch
    coef = _motion_coeffs(lib, tau.device)
    m = torch.arange(1, N_HARM + 1, dtype=torch.float64, device=tau.device)
    arg = (2.0 * math.pi * 0.5) * tau[:, None] * m[None, :]
    basis = torch.cat([torch.sin(arg), torch.cos(arg)], dim=1)                 # [n, 2H]
    r = torch.einsum("njkc,nk->njc", coef[clip_id], basis)
    q = _t_qexp_half(r)
    p = torch.stack([tau, torch.zeros_like(tau), ROOT_HEIGHT + 0.05 * torch.sin(2.0 * math.pi * tau)], dim=-1)
    return p, q


def _t_kinematics(skel: dict, root_p, q_l):
    import torch
    J = skel["J"]
    par = skel["parents"]
    off = torch.from_numpy(skel["offsets"].astype(np.float64)).to(q_l.device)
    p = [root_p]
    q = [q_l[:, 0]]
    for j in range(1, J):
        a = int(par[j])
        q.append(_t_qmul(q[a], q_l[:, j]))
        p.append(p[a] + _t_qrot(q[a], off[j].expand_as(p[a])))
    return torch.stack(p, dim=1), torch.stack(q, dim=1)


def synth_sim_state_torch(skel: dict, lib: dict, clip_id, t, step: int, wl: Workload,
                          seed: Optional[int] = None, env_base: int = 0):
    """Stand-in for the simulator: body states of n envs as one fp32 tensor [13J, n].

    clip_id (int64) and t (float64) are torch tensors; the result lives on their
    device.  Rows: 3J positions (x,y,z per body), 4J quaternions (w,x,y,z per
    body), 3J linear velocities, 3J angular velocities (world frame); element
    (c, e) at c*n + e.  State = analytic motion at each env's time plus
    joint-rotation noise N(0, sigma_q) rad, root noise N(0, sigma_root) m, and
    velocities from a central finite difference of the noise-free motion over
    1/fps plus N(0, sigma_vel) per component.  The noise is seeded per (seed,
    step, env_base) on the device in use.
    """
    import torch
    seed = wl.seed if seed is None else seed
    dev = t.device
    n = clip_id.shape[0]
    J = skel["J"]
    g = torch.Generator(device=dev)
    g.manual_seed((int(seed) * 1000003 + int(step)) * 1000003 + int(env_base) + 18)
    tau = t.to(torch.float64)
    cid = clip_id.to(torch.int64)
    h = 1.0 / wl.fps
    tau3 = torch.cat([tau - 0.5 * h, tau + 0.5 * h, tau])
    p3, q3 = _t_analytic_pose(lib, cid.repeat(3), tau3)
    noise = torch.randn((n, 9 * J + 3), generator=g, device=dev, dtype=torch.float64)
    q3[2 * n:] = _t_qmul(q3[2 * n:], _t_qexp_half(noise[:, :3 * J].reshape(n, J, 3) * wl.sigma_q))
    p3[2 * n:] += noise[:, 3 * J:3 * J + 3] * wl.sigma_root
    P3, Q3 = _t_kinematics(skel, p3, q3)
    lin = (P3[n:2 * n] - P3[:n]) / h + noise[:, 3 * J + 3:6 * J + 3].reshape(n, J, 3) * wl.sigma_vel
    ang = _t_qlog_rotvec(_t_qmul(Q3[n:2 * n], Q3[:n] * Q3.new_tensor([1.0, -1.0, -1.0, -1.0]))) / h
    ang = ang + noise[:, 6 * J + 3:].reshape(n, J, 3) * wl.sigma_vel
    out = torch.empty((13 * J, n), dtype=torch.float32, device=dev)
    out[0:3 * J] = P3[2 * n:].reshape(n, 3 * J).T
    out[3 * J:7 * J] = Q3[2 * n:].reshape(n, 4 * J).T
    out[7 * J:10 * J] = lin.reshape(n, 3 * J).T
    out[10 * J:13 * J] = ang.reshape(n, 3 * J).T
    return out


def synth_sim_state(skel: dict, lib: dict, clip_id: np.ndarray, t: np.ndarray, step: int,
                    wl: Workload, seed: Optional[int] = None, env_base: int = 0) -> np.ndarray:
    """numpy front end of synth_sim_state_torch (runs on the CPU)."""
    import torch
    out = synth_sim_state_torch(skel, lib, torch.from_numpy(np.ascontiguousarray(clip_id, np.int64)),
                                torch.from_numpy(np.ascontiguousarray(t, np.float64)), step, wl, seed, env_base)
    return out.numpy()


def split_sim(sim: np.ndarray, J: int):
    """Views (pos, quat, linvel, angvel) of a [13J, n] state array."""
    return sim[0:3 * J], sim[3 * J:7 * J], sim[7 * J:10 * J], sim[10 * J:13 * J]


# ----------------------------------------------------------------------------
# Policy weights: Kaiming-uniform W ~ U(+-sqrt(6/fan_in)), b ~ U(+-1/sqrt(fan_in)).
# ----------------------------------------------------------------------------
def round_to_bf16(x: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Round fp32 values to bf16 (nearest even). Returns (fp32 values, uint16 bits)."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32)
    r = ((u >> 16) & 1) + np.uint32(0x7FFF)
    bits = ((u + r) >> 16).astype(np.uint16)
    return (bits.astype(np.uint32) << 16).view(np.float32), bits


def make_policy_weights(dims: Sequence[int], dtype: str, seed: int = 0) -> dict:
    g = _rng(seed, 19)
    Ws, Wbits, bs = [], [], []
    for fan_in, fan_out in zip(dims[:-1], dims[1:]):
        W = g.uniform(-1.0, 1.0, size=(fan_out, fan_in)) * math.sqrt(6.0 / fan_in)
        b = g.uniform(-1.0, 1.0, size=fan_out) / math.sqrt(fan_in)
        W = W.astype(np.float32)
        if dtype == "bf16":
            W, bits = round_to_bf16(W)
            Wbits.append(bits)
        Ws.append(np.ascontiguousarray(W))
        bs.append(b.astype(np.float32))
    return dict(dims=tuple(int(d) for d in dims), dtype=dtype, W=Ws, W_bf16=Wbits, b=bs)


# ----------------------------------------------------------------------------
# Whole-rollout inputs.  `driver` is whichever implementation is being fed:
# it exposes the per-env (clip id, time) it holds and consumes one state array
# per step.  The generator never looks inside it.
# ----------------------------------------------------------------------------
def build_scene(wl: Workload) -> Tuple[dict, dict, dict]:
    skel = make_skeleton(wl.skeleton, wl.seed)
    lib = make_clip_library(skel["J"], wl.n_clips, wl.frames, wl.fps, wl.seed)
    pol = make_policy_weights(wl.mlp_dims, wl.mlp_dtype, wl.seed)
    return skel, lib, pol


def rollout_inputs(wl: Workload, skel: dict, lib: dict,
                   get_state: Callable[[], Tuple["np.ndarray", "np.ndarray"]],
                   consume: Callable[[int, "object"], None],
                   steps: Optional[int] = None, env_base: int = 0, device: str = "cpu") -> list:
    """Generate the per-step simulator states of a rollout.

    Before step s the driver reports each env's (clip id, time) as numpy arrays
    or torch tensors; the simulator stand-in produces the state one control
    interval later as a torch fp32 tensor [13J, n] on `device`; the driver then
    consumes it (which may reset some envs).  Returns the list of state tensors.
    """
    import torch
    sims = []
    for s in range(1, (wl.steps if steps is None else steps) + 1):
        cid, t = get_state()
        cid = torch.as_tensor(cid).to(device=device, dtype=torch.int64)
        t = torch.as_tensor(t).to(device=device, dtype=torch.float64)
        sim = synth_sim_state_torch(skel, lib, cid, t + wl.dt, s, wl, env_base=env_base)
        consume(s, sim)
        sims.append(sim)
    return sims


def shard_envs(n_total: int, world_size: int, rank: int) -> Tuple[int, int]:
    """Contiguous block partition of env ids: returns (first id, count) for a rank."""
    base, rem = divmod(n_total, world_size)
    first = rank * base + min(rank, rem)
    return first, base + (1 if rank < rem else 0)


# ----------------------------------------------------------------------------
# Rollout signals for the advantage estimator
# ----------------------------------------------------------------------------
def make_rollout_signals(T: int, N: int, seed: int = 0, p_term: float = 0.01, p_trunc: float = 0.01):
    """Seeded stand-ins for one rollout's per-step signals, time-major [T][N]: rewards U[0, 1) (the range
    of the imitation reward), critic outputs N(0, 3^2) for T + 1 observations, and flag bytes (bit 0
    terminated, bit 1 truncated) with the given per-step rates."""
    g = _rng(seed, 64, T, N)
    reward = g.random((T, N), dtype=np.float32)
    value = (3.0 * g.standard_normal((T + 1, N), dtype=np.float32)).astype(np.float32)
    flags = (g.random((T, N), dtype=np.float32) < p_term).astype(np.uint8)
    flags |= (g.random((T, N), dtype=np.float32) < p_trunc).astype(np.uint8) << 1
    return reward, value, flags


# ----------------------------------------------------------------------------
# One PPO minibatch for the loss kernel
# ----------------------------------------------------------------------------
def make_ppo_batch(M: int, A: int, seed: int = 0, drift: float = 0.05) -> dict:
    """Seeded stand-in for a minibatch some epochs into an update: the behaviour policy's means and
    log-stds, actions sampled from it with their log-probabilities, and a current policy that has
    drifted by `drift` (so a share of the probability ratios sits outside a 0.2 clip range);
    advantages N(0, 1) * 2 + 0.3, returns and values N(0, 3^2) with values near their old ones."""
    g = _rng(seed, 65, M, A)
    f32 = np.float32
    mean_old = g.standard_normal((M, A), dtype=f32)
    log_std_old = g.uniform(-2.0, -0.5, A).astype(f32)
    z = g.standard_normal((M, A), dtype=f32)
    action = (mean_old + np.exp(log_std_old) * z).astype(f32)
    logp_old = (-0.5 * (z.astype(np.float64) ** 2).sum(1) - log_std_old.astype(np.float64).sum()
                - 0.5 * A * math.log(2.0 * math.pi)).astype(f32)
    mean = (mean_old + drift * np.exp(log_std_old) * g.standard_normal((M, A), dtype=f32)).astype(f32)
    log_std = (log_std_old + 0.02 * g.standard_normal(A, dtype=f32)).astype(f32)
    value_old = (3.0 * g.standard_normal(M, dtype=f32)).astype(f32)
    value = (value_old + 0.3 * g.standard_normal(M, dtype=f32)).astype(f32)
    returns = (value_old + g.standard_normal(M, dtype=f32)).astype(f32)
    advantage = (2.0 * g.standard_normal(M, dtype=f32) + 0.3).astype(f32)
    return dict(mean=mean, log_std=log_std, action=action, logp_old=logp_old, mean_old=mean_old,
                log_std_old=log_std_old, advantage=advantage, value=value, value_old=value_old, returns=returns)
