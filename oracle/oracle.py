"""ctypes front end of the CPU oracle (oracle/im_oracle.c).  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg import
this module.  It compiles the C file with gcc on first use and shares nothing
with the CUDA library or its Python binding.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "im_oracle.c")
_OUT_DIR = os.path.join(_HERE, "_build")
_LIB = os.path.join(_OUT_DIR, "libim_oracle.so")
N_TERMS = 7


def build(force: bool = False) -> str:
    """Compile the oracle: gcc -O2, OpenMP over envs, no FMA contraction."""
    os.makedirs(_OUT_DIR, exist_ok=True)
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fPIC",
                               "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class RewardConfig(C.Structure):
    _fields_ = [("mode", C.c_int32), ("a", C.c_float * N_TERMS), ("w", C.c_float * N_TERMS),
                ("h_min", C.c_float), ("r_min", C.c_float)]


class EnvConfig(C.Structure):
    _fields_ = [("dt", C.c_float), ("seed_lo", C.c_uint32), ("seed_hi", C.c_uint32),
                ("reward", RewardConfig), ("write_back_reset", C.c_int32), ("grace_steps", C.c_int32),
                ("reset_noise_std", C.c_float), ("n_bins", C.c_int32), ("reset_cdf", C.c_void_p),
                ("stat_starts", C.c_void_p), ("stat_failures", C.c_void_p),
                ("n_future", C.c_int32), ("act_dim", C.c_int32), ("prev_action", C.c_void_p), ("ld_action", C.c_int64),
                ("cycle", C.c_void_p)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        vp, i32, u32, i64, f32, f64 = C.c_void_p, C.c_int32, C.c_uint32, C.c_int64, C.c_float, C.c_double
        L.orc_philox4x32_10.argtypes = [vp, vp, vp]
        L.orc_quat_mul.argtypes = [vp, vp, vp]
        L.orc_quat_rotate.argtypes = [vp, vp, vp]
        L.orc_quat_log.argtypes = [vp, vp]
        L.orc_geodesic_angle.argtypes = [vp]
        L.orc_geodesic_angle.restype = f64
        L.orc_slerp.argtypes = [vp, vp, f64, vp]
        L.orc_skeleton_create.argtypes = [i32, vp, vp, vp, vp, i32]
        L.orc_skeleton_create.restype = vp
        L.orc_skeleton_destroy.argtypes = [vp]
        L.orc_clips_create.argtypes = [vp, i32, vp, vp, vp, vp]
        L.orc_clips_create.restype = vp
        L.orc_clips_destroy.argtypes = [vp]
        L.orc_clips_set_cyclic.argtypes = [vp, vp]
        L.orc_clip_duration.argtypes = [vp, i32]
        L.orc_clip_duration.restype = f32
        L.orc_lookup_index.argtypes = [f32, f32, i32, vp, vp]
        L.orc_reference_state_flat.argtypes = [vp, vp, i32, f32] + [vp] * 7
        L.orc_reward.argtypes = [vp, vp]
        L.orc_reward.restype = f64
        L.orc_reset_draw.argtypes = [vp, vp, u32, u32, vp, vp]
        L.orc_env_reset_all.argtypes = [vp, vp, vp, i32, vp, u32, vp, vp, vp, vp, i64, i32]
        L.orc_env_step.argtypes = [vp, vp, vp, i32, vp, u32, vp, vp, vp, vp, vp, vp, vp, i64,
                                   vp, i64, vp, vp, vp, i32]
        L.orc_action_noise.argtypes = [u32, u32, u32, u32, i32, vp]
        L.orc_policy_forward.argtypes = [i32, vp, vp, vp, f64, u32, u32, u32, i32, vp, vp, i64,
                                         vp, vp, vp, vp, i32, i32]
        L.orc_policy_forward_std.argtypes = [i32, vp, vp, vp, f64, vp, u32, u32, u32, i32, vp, vp, i64,
                                             vp, vp, vp, vp, i32, i32]
        L.orc_round_bf16.argtypes = [f64]
        L.orc_round_bf16.restype = f64
        L.orc_error_terms_flat.argtypes = [vp, vp, i32, f32, vp, vp, vp, vp, vp]
        L.orc_openmp_enabled.restype = i32
        L.orc_reset_state_flat.argtypes = [vp, vp, vp, u32, u32, i32, f32, vp, vp, vp, vp, vp]
        L.orc_reset_cdf.argtypes = [i32, vp, vp]
        L.orc_reset_cdf.restype = i32
        L.orc_ppo_loss.argtypes = [vp, i64, i32] + [vp] * 7 + [f64, f64] + [vp] * 7
        L.orc_moments.argtypes = [vp, i64, vp, vp]
        L.orc_adam_step.argtypes = [i64, vp, vp, vp, vp, f64, f64, f64, f64, i32, f64]
        L.orc_grad_scale.argtypes = [i32, vp, vp, f64]
        L.orc_grad_scale.restype = f64
        L.orc_adaptive_lr.argtypes = [f64] * 5
        L.orc_adaptive_lr.restype = f64
        L.orc_mlp_backward.argtypes = [i32, vp, vp, vp, i32, vp, i64, vp, vp, vp, i32]
        L.orc_gae.argtypes = [i32, i32, i64, vp, vp, vp, f64, f64, i32, vp, vp]
        _lib = L
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _f64(x) -> np.ndarray:
    return np.ascontiguousarray(x, np.float64)


# ---------------------------------------------------------------- small pieces
def philox(ctr: Sequence[int], key: Sequence[int]) -> np.ndarray:
    c = np.asarray(ctr, np.uint32)
    k = np.asarray(key, np.uint32)
    out = np.empty(4, np.uint32)
    lib().orc_philox4x32_10(_p(c), _p(k), _p(out))
    return out


def quat_mul(a, b) -> np.ndarray:
    a, b, out = _f64(a), _f64(b), np.empty(4)
    lib().orc_quat_mul(_p(a), _p(b), _p(out))
    return out


def quat_rotate(q, v) -> np.ndarray:
    q, v, out = _f64(q), _f64(v), np.empty(3)
    lib().orc_quat_rotate(_p(q), _p(v), _p(out))
    return out


def quat_log(q) -> np.ndarray:
    q, out = _f64(q), np.empty(3)
    lib().orc_quat_log(_p(q), _p(out))
    return out


def geodesic_angle(q) -> float:
    q = _f64(q)
    return float(lib().orc_geodesic_angle(_p(q)))


def slerp(q0, q1, alpha: float) -> np.ndarray:
    q0, q1, out = _f64(q0), _f64(q1), np.empty(4)
    lib().orc_slerp(_p(q0), _p(q1), float(alpha), _p(out))
    return out


def lookup_index(t: float, fps: float, K: int):
    k = np.zeros(1, np.int32)
    a = np.zeros(1, np.float64)
    lib().orc_lookup_index(np.float32(t), np.float32(fps), int(K), _p(k), _p(a))
    return int(k[0]), float(a[0])


def action_noise(seed: int, env: int, step: int, A: int) -> np.ndarray:
    z = np.zeros(A + 4)
    lib().orc_action_noise(seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF, env, step, A, _p(z))
    return z[:A]


def make_env_config(dt: float, seed: int, reward: dict, h_min: float, r_min: float = -np.inf,
                    write_back_reset: bool = False, grace_steps: int = 0, reset_noise_std: float = 0.0) -> EnvConfig:
    rc = RewardConfig(mode=int(reward["mode"]), h_min=np.float32(h_min), r_min=np.float32(r_min))
    for k in range(N_TERMS):
        rc.a[k] = reward["a"][k]
        rc.w[k] = reward["w"][k]
    return EnvConfig(dt=np.float32(dt), seed_lo=seed & 0xFFFFFFFF, seed_hi=(seed >> 32) & 0xFFFFFFFF,
                     reward=rc, write_back_reset=int(write_back_reset), grace_steps=int(grace_steps),
                     reset_noise_std=np.float32(reset_noise_std))


def reward_from_terms(reward: dict, e) -> float:
    cfg = make_env_config(1.0 / 30, 0, reward, 0.0)
    e = _f64(e)
    return float(lib().orc_reward(C.byref(cfg.reward), _p(e)))


# ---------------------------------------------------------------- handles
class Skeleton:
    def __init__(self, parents, offsets, masses=None, ee_ids=None):
        self.parents = np.ascontiguousarray(parents, np.int32)
        self.J = int(self.parents.shape[0])
        off = np.ascontiguousarray(offsets, np.float32)
        m = None if masses is None else np.ascontiguousarray(masses, np.float32)
        ee = None if ee_ids is None else np.ascontiguousarray(ee_ids, np.int32)
        # end effectors: the given bodies, else the bodies without children
        self.ee_ids = sorted(int(e) for e in ee) if ee is not None else \
            [j for j in range(self.J) if j not in set(int(p) for p in self.parents)]
        self.n_ee = len(self.ee_ids)
        self.h = lib().orc_skeleton_create(self.J, _p(self.parents), _p(off), _p(m), _p(ee),
                                           0 if ee is None else int(ee.shape[0]))
        if not self.h:
            raise ValueError("invalid skeleton")

    def __del__(self):
        if getattr(self, "h", None) and _lib is not None:
            _lib.orc_skeleton_destroy(self.h)
            self.h = None


class Clips:
    def __init__(self, skel: Skeleton, n_frames, fps, root_pos, local_quat):
        self.skel = skel
        self.n_frames = np.ascontiguousarray(n_frames, np.int32)
        self.fps = np.ascontiguousarray(fps, np.float32)
        self.C = int(self.n_frames.shape[0])
        rp = np.ascontiguousarray(root_pos, np.float32)
        lq = np.ascontiguousarray(local_quat, np.float32)
        assert rp.shape == (int(self.n_frames.sum()), 3)
        assert lq.shape == (int(self.n_frames.sum()), skel.J, 4)
        self.h = lib().orc_clips_create(skel.h, self.C, _p(self.n_frames), _p(self.fps), _p(rp), _p(lq))

    def duration(self, clip: int) -> np.float32:
        return np.float32(lib().orc_clip_duration(self.h, int(clip)))

    def set_cyclic(self, flags) -> None:
        """flags: one byte per clip (non-zero: the clip is played in a loop), or None to clear all."""
        f = None if flags is None else np.ascontiguousarray(flags, np.uint8)
        assert f is None or f.shape == (self.C,)
        self.cyclic = np.zeros(self.C, np.uint8) if f is None else f.copy()
        lib().orc_clips_set_cyclic(self.h, _p(f))

    def __del__(self):
        if getattr(self, "h", None) and _lib is not None:
            _lib.orc_clips_destroy(self.h)
            self.h = None


def reference_state(skel: Skeleton, clips: Clips, clip: int, t: float) -> dict:
    J = skel.J
    out = dict(p=np.empty((J, 3)), q=np.empty((J, 4)), v=np.empty((J, 3)), w=np.empty((J, 3)),
               ql=np.empty((J, 4)), wl=np.empty((J, 3)), com=np.empty(3))
    lib().orc_reference_state_flat(skel.h, clips.h, int(clip), np.float32(t), _p(out["p"]), _p(out["q"]),
                                   _p(out["v"]), _p(out["w"]), _p(out["ql"]), _p(out["wl"]), _p(out["com"]))
    return out


def error_terms(skel: Skeleton, clips: Clips, clip: int, t: float, p, q, v, w) -> np.ndarray:
    e = np.empty(N_TERMS)
    p, q, v, w = _f64(p), _f64(q), _f64(v), _f64(w)
    lib().orc_error_terms_flat(skel.h, clips.h, int(clip), np.float32(t), _p(p), _p(q), _p(v), _p(w), _p(e))
    return e


def reset_draw(clips: Clips, cfg: EnvConfig, env: int, step: int):
    c = np.zeros(1, np.int32)
    t = np.zeros(1, np.float32)
    lib().orc_reset_draw(clips.h, C.byref(cfg), env, step, _p(c), _p(t))
    return int(c[0]), np.float32(t[0])


class Env:
    """Per-env state (clip id, time, episode length) plus the step functions."""

    def __init__(self, skel: Skeleton, clips: Clips, cfg: EnvConfig, n_envs: int,
                 env_ids: Optional[np.ndarray] = None, n_threads: Optional[int] = None):
        self.skel, self.clips, self.cfg, self.n = skel, clips, cfg, int(n_envs)
        self.env_ids = (np.arange(n_envs, dtype=np.uint32) if env_ids is None
                        else np.ascontiguousarray(env_ids, np.uint32))
        self.clip_id = np.zeros(self.n, np.int32)
        self.t = np.zeros(self.n, np.float32)
        self.ep_len = np.zeros(self.n, np.int32)
        self.cycle = np.zeros(self.n, np.int32)          # cycles completed on a cyclic clip (0 elsewhere)
        self.cfg.cycle = self.cycle.ctypes.data
        self.D = 24 * skel.J + 1
        self.n_threads = int(n_threads or os.cpu_count() or 1)

    def set_reset_bins(self, n_bins: int, weights) -> None:
        """Adaptive episode initialisation: weights [C, n_bins] over (clip, phase bin)."""
        w = np.ascontiguousarray(weights, np.float32)
        assert w.shape == (self.clips.C, n_bins)
        self.reset_cdf = reset_cdf(w.ravel())
        self.stat_starts = np.zeros(w.size, np.uint32)
        self.stat_failures = np.zeros(w.size, np.uint32)
        self.cfg.n_bins = int(n_bins)
        self.cfg.reset_cdf = self.reset_cdf.ctypes.data
        self.cfg.stat_starts = self.stat_starts.ctypes.data
        self.cfg.stat_failures = self.stat_failures.ctypes.data

    def adapt_reset_bins(self, floor_weight: float, clear: bool = True) -> np.ndarray:
        """Adaptive episode initialisation from the failure counts (Section 6 names adaptive sampling after
        [Won 2019/2020] without the rule; this build's: bins where more episodes ended early are started
        more often): weight of (clip, bin) i = fl32(fl32(failures_i) + floor_weight), then the cumulative
        table of those weights replaces the current one; the counts are cleared if asked.  Returns the weights."""
        w = (self.stat_failures.astype(np.float32) + np.float32(floor_weight)).astype(np.float32)
        self.reset_cdf = reset_cdf(w)
        self.cfg.reset_cdf = self.reset_cdf.ctypes.data
        if clear:
            self.stat_starts[:] = 0
            self.stat_failures[:] = 0
        return w

    def set_obs_extension(self, n_future: int = 1, prev_action: Optional[np.ndarray] = None) -> int:
        """Extended observation: end-effector targets of reference frames 2 .. n_future, then the previous action
        (fp32 [n, A]; the array is read by later steps, so the caller updates it in place).  Returns the width."""
        self.prev_action = None if prev_action is None else prev_action
        A = 0
        if prev_action is not None:
            assert prev_action.dtype == np.float32 and prev_action.shape[0] == self.n and prev_action.flags.c_contiguous
            A = prev_action.shape[1]
            self.cfg.prev_action = prev_action.ctypes.data
            self.cfg.ld_action = A
        self.cfg.n_future = int(n_future)
        self.cfg.act_dim = A
        self.D = 24 * self.skel.J + 1 + (int(n_future) - 1) * 9 * self.skel.n_ee + A
        return self.D

    def reset_all(self, step: int = 0) -> np.ndarray:
        obs = np.zeros((self.n, self.D))
        lib().orc_env_reset_all(self.skel.h, self.clips.h, C.byref(self.cfg), self.n, _p(self.env_ids), step,
                                _p(self.clip_id), _p(self.t), _p(self.ep_len), _p(obs), self.D,
                                self.n_threads)
        return obs

    def step(self, step: int, sim: np.ndarray, want_terms: bool = True) -> dict:
        """sim: fp32 [13J, n] (positions, quaternions, linear, angular velocities)."""
        J = self.skel.J
        assert sim.dtype == np.float32 and sim.shape == (13 * J, self.n) and sim.flags.c_contiguous
        pos, quat, lin, ang = sim[0:3 * J], sim[3 * J:7 * J], sim[7 * J:10 * J], sim[10 * J:13 * J]
        obs = np.zeros((self.n, self.D))
        reward = np.zeros(self.n)
        flags = np.zeros(self.n, np.uint8)
        terms = np.zeros((N_TERMS, self.n)) if want_terms else None
        lib().orc_env_step(self.skel.h, self.clips.h, C.byref(self.cfg), self.n, _p(self.env_ids), step,
                           _p(self.clip_id), _p(self.t), _p(self.ep_len),
                           _p(pos), _p(quat), _p(lin), _p(ang), self.n,
                           _p(obs), self.D, _p(reward), _p(flags), _p(terms), self.n_threads)
        return dict(obs=obs, reward=reward, flags=flags, terms=terms)


def round_bf16(x: float) -> float:
    return float(lib().orc_round_bf16(float(x)))


def policy_forward(dims, W, b, sigma: float, seed: int, step: int, obs: np.ndarray,
                   env_ids: Optional[np.ndarray] = None, n_threads: Optional[int] = None,
                   bf16_operands: bool = False, log_std: Optional[np.ndarray] = None) -> dict:
    """obs: fp64 [n, >=dims[0]].  W[l]: fp32 [dims[l+1], dims[l]] (bf16 weights widened exactly).
    bf16_operands: observation and hidden activations are rounded to bf16 before each layer.
    log_std: fp32 [A], per-dimension standard deviation exp(log_std) instead of the scalar sigma."""
    nl = len(dims) - 1
    n = obs.shape[0]
    obs = _f64(obs)
    A = int(dims[-1])
    ids = np.arange(n, dtype=np.uint32) if env_ids is None else np.ascontiguousarray(env_ids, np.uint32)
    Wc = [np.ascontiguousarray(w, np.float32) for w in W]
    bc = [np.ascontiguousarray(x, np.float32) for x in b]
    for l in range(nl):
        assert Wc[l].shape == (dims[l + 1], dims[l]) and bc[l].shape == (dims[l + 1],)
    Wp = (C.c_void_p * nl)(*[w.ctypes.data for w in Wc])
    bp = (C.c_void_p * nl)(*[x.ctypes.data for x in bc])
    d = np.asarray(dims, np.int32)
    mean = np.zeros((n, A))
    action = np.zeros((n, A))
    logp = np.zeros(n)
    z = np.zeros((n, A))
    ls = None if log_std is None else np.ascontiguousarray(log_std, np.float32)
    assert ls is None or ls.shape == (A,)
    lib().orc_policy_forward_std(nl, _p(d), C.cast(Wp, C.c_void_p), C.cast(bp, C.c_void_p), float(sigma), _p(ls),
                             seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF, step, n, _p(ids),
                             _p(obs), obs.shape[1], _p(mean), _p(action), _p(logp), _p(z),
                             int(n_threads or os.cpu_count() or 1), int(bool(bf16_operands)))
    return dict(mean=mean, action=action, logp=logp, z=z)


def gae(reward: np.ndarray, value: np.ndarray, flags: np.ndarray, gamma: float, lam: float,
        bootstrap_truncated: bool = True):
    """reward [T, N] fp32, value [T+1, N] fp32, flags [T, N] uint8 -> (advantage, return) fp64 [T, N]."""
    reward = np.ascontiguousarray(reward, np.float32)
    value = np.ascontiguousarray(value, np.float32)
    flags = np.ascontiguousarray(flags, np.uint8)
    T, N = reward.shape
    assert value.shape == (T + 1, N) and flags.shape == (T, N)
    adv = np.zeros((T, N))
    ret = np.zeros((T, N))
    lib().orc_gae(T, N, N, _p(reward), _p(value), _p(flags), float(gamma), float(lam),
                  int(bool(bootstrap_truncated)), _p(adv), _p(ret))
    return adv, ret


def reset_state(skel: Skeleton, clips: Clips, cfg: EnvConfig, env: int, step: int, clip: int, t: float) -> dict:
    """State an env reset at (clip, t) with counter (env, step) starts from (motion randomisation applied)."""
    J = skel.J
    out = {k: np.zeros((J, n)) for k, n in (("p", 3), ("q", 4), ("v", 3), ("w", 3), ("ql", 4))}
    lib().orc_reset_state_flat(skel.h, clips.h, C.byref(cfg), env, step, clip, np.float32(t),
                               _p(out["p"]), _p(out["q"]), _p(out["v"]), _p(out["w"]), _p(out["ql"]))
    return out


def reset_cdf(weights) -> np.ndarray:
    """Cumulative thresholds (uint64, in [0, 2^32]) of a flat weight table."""
    w = np.ascontiguousarray(weights, np.float32).ravel()
    T = np.zeros(w.size, np.uint64)
    if lib().orc_reset_cdf(w.size, _p(w), _p(T)) != 0:
        raise ValueError("weights must be finite, non-negative and not all zero")
    return T


class PpoConfig(C.Structure):
    _fields_ = [("clip", C.c_float), ("value_coef", C.c_float), ("entropy_coef", C.c_float),
                ("clip_value_loss", C.c_int32)]


def moments(x) -> tuple:
    """(mean, 1 / (std + 1e-8)) with the n - 1 divisor."""
    x = np.ascontiguousarray(x, np.float32).ravel()
    m, r = C.c_double(), C.c_double()
    lib().orc_moments(_p(x), x.size, C.byref(m), C.byref(r))
    return m.value, r.value


def ppo_loss(batch: dict, clip: float, value_coef: float, entropy_coef: float, clip_value_loss: bool,
             adv_mean: float = 0.0, adv_rstd: float = 1.0) -> dict:
    """batch: mean, action, mean_old [M, A]; log_std, log_std_old [A]; logp_old, advantage, value,
    value_old, returns [M] (all read as fp32).  Returns d_mean, d_log_std, d_value, summary (fp64)."""
    f = {k: np.ascontiguousarray(v, np.float32) for k, v in batch.items()}
    M, A = f["mean"].shape
    cfg = PpoConfig(np.float32(clip), np.float32(value_coef), np.float32(entropy_coef), int(bool(clip_value_loss)))
    out = dict(d_mean=np.zeros((M, A)), d_log_std=np.zeros(A), d_value=np.zeros(M), summary=np.zeros(6))
    lib().orc_ppo_loss(C.byref(cfg), M, A, _p(f["mean"]), _p(f["log_std"]), _p(f["action"]), _p(f["logp_old"]),
                       _p(f["mean_old"]), _p(f["log_std_old"]), _p(f["advantage"]), float(adv_mean), float(adv_rstd),
                       _p(f["value"]), _p(f["value_old"]), _p(f["returns"]), _p(out["d_mean"]),
                       _p(out["d_log_std"]), _p(out["d_value"]), _p(out["summary"]))
    return out


def adam_step(param, grad, m, v, lr: float, t: int, b1: float = 0.9, b2: float = 0.999, eps: float = 1e-8,
              grad_scale: float = 1.0):
    """In-place Adam step on contiguous fp32 numpy arrays (param, m, v are updated)."""
    for a in (param, grad, m, v):
        assert a.dtype == np.float32 and a.flags.c_contiguous and a.size == param.size
    lib().orc_adam_step(param.size, _p(param), _p(grad), _p(m), _p(v), float(lr), float(b1), float(b2), float(eps),
                        int(t), float(grad_scale))


def grad_scale(grads, max_norm: float) -> float:
    """min(1, max_norm / (global L2 norm + 1e-6)) over a list of fp32 arrays."""
    gs = [np.ascontiguousarray(g, np.float32).ravel() for g in grads]
    ptrs = (C.c_void_p * len(gs))(*[g.ctypes.data for g in gs])
    sizes = np.asarray([g.size for g in gs], np.int64)
    return float(lib().orc_grad_scale(len(gs), C.cast(ptrs, C.c_void_p), _p(sizes), float(max_norm)))


def adaptive_lr(lr: float, kl: float, kl_target: float, lr_min: float = 1e-5, lr_max: float = 1e-2) -> float:
    return float(lib().orc_adaptive_lr(float(lr), float(kl), float(kl_target), float(lr_min), float(lr_max)))


def mlp_backward(dims, W, b, obs: np.ndarray, g_out: np.ndarray, bf16_operands: bool = False):
    """Gradients (dW list, db list, fp64) of a loss with dL/d(output) = g_out [n, A] for the MLP on obs [n, >=dims[0]]."""
    nl = len(dims) - 1
    obs = _f64(obs)
    g_out = _f64(g_out)
    n = obs.shape[0]
    assert g_out.shape == (n, dims[-1])
    Wc = [np.ascontiguousarray(w, np.float32) for w in W]
    bc = [np.ascontiguousarray(x, np.float32) for x in b]
    Wp = (C.c_void_p * nl)(*[w.ctypes.data for w in Wc])
    bp = (C.c_void_p * nl)(*[x.ctypes.data for x in bc])
    d = np.asarray(dims, np.int32)
    dW = np.zeros(sum(int(dims[l]) * int(dims[l + 1]) for l in range(nl)))
    db = np.zeros(sum(int(dims[l + 1]) for l in range(nl)))
    lib().orc_mlp_backward(nl, _p(d), C.cast(Wp, C.c_void_p), C.cast(bp, C.c_void_p), n, _p(obs), obs.shape[1],
                           _p(g_out), _p(dW), _p(db), int(bool(bf16_operands)))
    outW, outb, wo, bo = [], [], 0, 0
    for l in range(nl):
        k, m = int(dims[l]), int(dims[l + 1])
        outW.append(dW[wo:wo + m * k].reshape(m, k)); wo += m * k
        outb.append(db[bo:bo + m]); bo += m
    return outW, outb
