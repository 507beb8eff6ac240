"""Thin ctypes binding over the C-ABI CUDA library (include/im.h).

Argument marshalling only: every step of the path runs in the library's
kernels.  torch supplies device memory and the CUDA stream.  The shared object
is loaded on first use; if it is missing the calls raise -- there is no
fallback implementation.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# IM_B200_LIB selects another build of the library (e.g. the bounds-checked libim_b200_debug.so)
LIB_PATH = os.environ.get("IM_B200_LIB") or os.path.join(_HERE, "_build", "libim_b200.so")
N_TERMS = 7
MAX_LAYERS = 8

EXPORTS = [
    "im_status_string", "im_create_skeleton", "im_destroy_skeleton", "im_load_clips", "im_destroy_clips",
    "im_env_create", "im_env_destroy", "im_env_reset_all", "im_env_step", "im_env_get_state",
    "im_env_set_state", "im_load_policy", "im_destroy_policy", "im_policy_forward",
    "im_env_reset_all_host", "im_step_host", "im_poll_device_status", "im_launch_count",
    "im_policy_forward_noalloc", "im_env_attach_policy", "im_policy_forward_staged",
    "im_value_forward", "im_value_forward_staged", "im_gae", "im_env_set_reset_bins", "im_env_get_reset_stats",
    "im_env_step_aos", "im_policy_set_log_std", "im_ppo_workspace_bytes", "im_moments", "im_ppo_loss",
    "im_adam_step", "im_grad_scale", "im_adaptive_lr", "im_policy_layer_buffers",
    "im_gemm_bf16", "im_gemm_bf16_f32out", "im_transpose_bf16", "im_f32_to_bf16_padded",
    "im_colsum_f32", "im_sum_slices_bf16_to_f32",
    "im_trainer_create", "im_trainer_destroy", "im_trainer_forward", "im_trainer_backward", "im_trainer_step",
    "im_trainer_push_to_policy", "im_trainer_tensor", "im_trainer_set_step_count", "im_trainer_dw_slices",
    "im_ppo_updater_create", "im_ppo_updater_destroy", "im_ppo_update", "im_ppo_update_rollout", "im_ppo_updater_tensor",
    "im_ppo_updater_set_step_count",
    "im_copy_f32", "im_gemm_bf16_tn", "im_gather_rows_f32", "im_gemm_bf16_dgrad", "im_env_set_obs_extension", "im_env_adapt_reset_bins", "im_debug_math", "im_debug_set_wait", "im_env_set_summary", "im_clips_set_cyclic",
    "im_env_get_cycles", "im_env_set_cycles", "im_env_set_aos_staging",
]


class RewardConfig(C.Structure):
    _fields_ = [("mode", C.c_int32), ("a", C.c_float * N_TERMS), ("w", C.c_float * N_TERMS),
                ("h_min", C.c_float), ("r_min", C.c_float)]


class EnvConfig(C.Structure):
    _fields_ = [("n_envs", C.c_int32), ("env_id_base", C.c_uint32), ("dt", C.c_float), ("seed", C.c_uint64),
                ("reward", RewardConfig), ("ld_obs", C.c_int32), ("write_back_reset", C.c_int32),
                ("grace_steps", C.c_int32), ("reset_noise_std", C.c_float)]


class AosArray(C.Structure):
    _fields_ = [("base", C.c_void_p), ("env_stride", C.c_int64), ("body_stride", C.c_int32)]


class BodyStateAos(C.Structure):
    _fields_ = [("pos", AosArray), ("quat", AosArray), ("linvel", AosArray), ("angvel", AosArray)]


class BodyState(C.Structure):
    _fields_ = [("pos", C.c_void_p), ("quat", C.c_void_p), ("linvel", C.c_void_p), ("angvel", C.c_void_p),
                ("comp_stride", C.c_int64)]


class GaeConfig(C.Structure):
    _fields_ = [("gamma", C.c_float), ("lam", C.c_float), ("bootstrap_truncated", C.c_int32)]


class PpoConfig(C.Structure):
    _fields_ = [("clip", C.c_float), ("value_coef", C.c_float), ("entropy_coef", C.c_float),
                ("clip_value_loss", C.c_int32)]


class PpoBatch(C.Structure):
    _fields_ = [(k, C.c_void_p) for k in ("mean", "log_std", "action", "logp_old", "mean_old", "log_std_old",
                                          "advantage", "adv_moments", "value", "value_old", "returns")]


class AdamConfig(C.Structure):
    _fields_ = [("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float)]


class PpoUpdateConfig(C.Structure):
    _fields_ = [("lr", C.c_float), ("clip", C.c_float), ("value_coef", C.c_float), ("entropy_coef", C.c_float),
                ("clip_value_loss", C.c_int32), ("max_grad_norm", C.c_float), ("kl_target", C.c_float),
                ("lr_min", C.c_float), ("lr_max", C.c_float), ("normalize_advantage", C.c_int32), ("adam", AdamConfig)]


class PpoMinibatch(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("action", "mean_old", "log_std_old", "logp_old", "advantage", "value_old", "returns")]


class RolloutView(C.Structure):
    _fields_ = [("T", C.c_int32), ("N", C.c_int32), ("A", C.c_int32), ("ld_obs", C.c_int32)] + \
               [(n, C.c_void_p) for n in ("obs", "action", "mean", "logp", "advantage", "returns", "value")]


class PolicyConfig(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("dims", C.c_int32 * (MAX_LAYERS + 1)), ("dtype", C.c_int32),
                ("sigma", C.c_float), ("seed", C.c_uint64), ("env_id_base", C.c_uint32),
                ("max_batch", C.c_int32), ("impl", C.c_int32)]


class ImError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__("%s: %s (status %d)" % (what, _lib.im_status_string(status).decode(), status))
        self.status = status


_lib = None


def load():
    """Loads the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("CUDA library not built: %s is missing (run python -m paper_2609_09821_b200.build)"
                               % LIB_PATH)
        L = C.CDLL(LIB_PATH)
        vp, i32, u32, u64 = C.c_void_p, C.c_int32, C.c_uint32, C.c_uint64
        L.im_status_string.argtypes = [i32]
        L.im_status_string.restype = C.c_char_p
        L.im_create_skeleton.argtypes = [i32, vp, vp, vp, vp, i32, C.POINTER(vp)]
        L.im_destroy_skeleton.argtypes = [vp]
        L.im_load_clips.argtypes = [vp, i32, vp, vp, vp, vp, C.POINTER(vp)]
        L.im_destroy_clips.argtypes = [vp]
        L.im_env_create.argtypes = [vp, vp, C.POINTER(EnvConfig), vp, C.POINTER(vp)]
        L.im_env_destroy.argtypes = [vp]
        L.im_env_reset_all.argtypes = [vp, u32, vp]
        L.im_env_step.argtypes = [vp, u32, C.POINTER(BodyState), vp, vp, vp, vp]
        L.im_env_step_aos.argtypes = [vp, u32, C.POINTER(BodyStateAos), vp, vp, vp, vp]
        L.im_env_get_state.argtypes = [vp, vp, vp, vp]
        L.im_env_set_state.argtypes = [vp, vp, vp, vp]
        L.im_load_policy.argtypes = [C.POINTER(PolicyConfig), vp, vp, vp, C.POINTER(vp)]
        L.im_destroy_policy.argtypes = [vp]
        L.im_policy_forward.argtypes = [vp, u32, i32, vp, i32, vp, vp, vp]
        L.im_env_reset_all_host.argtypes = [vp, u32]
        L.im_step_host.argtypes = [vp, vp, u32, vp, vp, vp, vp]
        L.im_poll_device_status.argtypes = [vp, vp, C.POINTER(u32)]
        L.im_launch_count.restype = u64
        L.im_env_attach_policy.argtypes = [vp, vp]
        L.im_policy_forward_staged.argtypes = [vp, u32, i32, vp, vp, vp]
        L.im_policy_forward_noalloc.argtypes = [i32, vp, vp, vp, C.c_float, u64, u32, u32, i32, vp, i32, vp, vp, vp, vp]
        L.im_env_set_reset_bins.argtypes = [vp, i32, vp]
        L.im_env_get_reset_stats.argtypes = [vp, vp, vp, i32]
        L.im_policy_set_log_std.argtypes = [vp, vp]
        L.im_ppo_workspace_bytes.restype = C.c_size_t
        L.im_moments.argtypes = [vp, C.c_int64, vp, vp, vp]
        L.im_ppo_loss.argtypes = [C.POINTER(PpoConfig), C.c_int64, i32, C.POINTER(PpoBatch), vp, vp, vp, vp, vp, vp]
        L.im_adam_step.argtypes = [C.POINTER(AdamConfig), i32, C.c_int64, vp, vp, vp, vp, vp, vp, vp, i32, i32, vp]
        L.im_grad_scale.argtypes = [i32, vp, vp, C.c_float, vp, vp, vp]
        L.im_adaptive_lr.argtypes = [vp, vp, C.c_float, C.c_float, C.c_float, vp]
        L.im_policy_layer_buffers.argtypes = [vp, i32, C.POINTER(vp), C.POINTER(i32), C.POINTER(vp)]
        i64 = C.c_int64
        L.im_gemm_bf16.argtypes = [vp, i64, vp, i64, vp, i64, i32, i32, i32, vp, i32, vp, vp]
        L.im_gemm_bf16_tn.argtypes = [vp, i64, vp, i64, vp, i64, i32, i32, i32, i32, i32, vp, vp]
        L.im_sum_slices_bf16_to_f32.argtypes = [vp, i64, i64, i32, i32, i32, vp, vp]
        L.im_gemm_bf16_f32out.argtypes = [vp, i64, vp, i64, vp, i32, i32, i32, vp, vp, vp]
        L.im_transpose_bf16.argtypes = [vp, i64, i32, i32, vp, i64, vp]
        L.im_f32_to_bf16_padded.argtypes = [vp, i64, i32, i32, vp, i32, vp]
        L.im_env_adapt_reset_bins.argtypes = [vp, C.c_float, i32]
        L.im_debug_math.argtypes = [i32, i32, vp, vp, vp]
        L.im_debug_set_wait.argtypes = [u64, i32]
        L.im_env_set_summary.argtypes = [vp, vp]
        L.im_clips_set_cyclic.argtypes = [vp, vp]
        L.im_env_get_cycles.argtypes = [vp, vp]
        L.im_env_set_aos_staging.argtypes = [vp, i32]
        L.im_env_set_cycles.argtypes = [vp, vp]
        L.im_env_set_obs_extension.argtypes = [vp, i32, i32, vp, i32]
        L.im_gemm_bf16_dgrad.argtypes = [vp, i64, vp, i64, vp, i64, i32, i32, i32, vp, i64, vp, i32, vp, vp]
        L.im_trainer_create.argtypes = [i32, vp, vp, vp, i32, vp, C.POINTER(vp)]
        L.im_trainer_destroy.argtypes = [vp]
        L.im_trainer_destroy.restype = None
        L.im_trainer_forward.argtypes = [vp, i32]
        L.im_trainer_backward.argtypes = [vp, vp, i32]
        L.im_trainer_step.argtypes = [vp, C.POINTER(AdamConfig), vp, vp]
        L.im_trainer_push_to_policy.argtypes = [vp, vp]
        L.im_trainer_tensor.argtypes = [vp, i32, i32, C.POINTER(vp), C.POINTER(i64), C.POINTER(i64), C.POINTER(i64), C.POINTER(i32)]
        L.im_trainer_set_step_count.argtypes = [vp, i32]
        L.im_trainer_dw_slices.argtypes = [i32, i32, i64, i32, i32]
        L.im_trainer_dw_slices.restype = i32
        L.im_ppo_updater_create.argtypes = [vp, vp, vp, C.POINTER(PpoUpdateConfig), C.POINTER(vp)]
        L.im_ppo_updater_destroy.argtypes = [vp]
        L.im_ppo_updater_destroy.restype = None
        L.im_ppo_update.argtypes = [vp, i32, C.POINTER(PpoMinibatch)]
        L.im_ppo_update_rollout.argtypes = [vp, C.POINTER(RolloutView), i32, i32, vp]
        L.im_ppo_updater_tensor.argtypes = [vp, i32, C.POINTER(vp), C.POINTER(i64)]
        L.im_ppo_updater_set_step_count.argtypes = [vp, i32]
        L.im_gather_rows_f32.argtypes = [vp, i64, vp, i64, i32, i32, vp, i32, i32, vp, vp]
        L.im_copy_f32.argtypes = [vp, vp, i64, vp]
        L.im_colsum_f32.argtypes = [vp, i64, i64, i32, vp, vp, C.c_size_t, vp]
        L.im_value_forward.argtypes = [vp, i32, vp, i32, vp]
        L.im_value_forward_staged.argtypes = [vp, vp, i32, vp]
        L.im_gae.argtypes = [C.POINTER(GaeConfig), i32, i32, C.c_int64, vp, vp, vp, vp, vp, vp]
        for name in EXPORTS:
            if name not in ("im_status_string", "im_launch_count", "im_ppo_workspace_bytes") \
                    and not name.startswith("im_destroy") \
                    and name != "im_env_destroy":
                getattr(L, name).restype = i32
        _lib = L
    return _lib


def _check(status: int, what: str):
    if status != 0:
        raise ImError(status, what)


def _np(a, dtype):
    return None if a is None else np.ascontiguousarray(a, dtype)


def _ptr(a):
    if a is None:
        return None
    if isinstance(a, np.ndarray):
        return a.ctypes.data_as(C.c_void_p)
    return C.c_void_p(a.data_ptr())          # torch tensor


def launch_count() -> int:
    return int(load().im_launch_count())


class Skeleton:
    def __init__(self, parents, offsets, masses=None, ee_ids=None):
        L = load()
        par = _np(parents, np.int32)
        off = _np(offsets, np.float32)
        m = _np(masses, np.float32)
        ee = _np(ee_ids, np.int32)
        self.J = int(par.shape[0])
        # end effectors: the given bodies, else the leaves of the tree
        self.n_ee = int(ee.shape[0]) if ee is not None else self.J - len(set(int(x) for x in par if x >= 0))
        self.h = C.c_void_p()
        _check(L.im_create_skeleton(self.J, _ptr(par), _ptr(off), _ptr(m), _ptr(ee),
                                    0 if ee is None else int(ee.shape[0]), C.byref(self.h)), "im_create_skeleton")

    def __del__(self):
        if getattr(self, "h", None) and _lib is not None:
            _lib.im_destroy_skeleton(self.h)
            self.h = None


class Clips:
    def __init__(self, skel: Skeleton, n_frames, fps, root_pos, local_quat):
        L = load()
        self.skel = skel
        nf = _np(n_frames, np.int32)
        f = _np(fps, np.float32)
        rp = _np(root_pos, np.float32)
        lq = _np(local_quat, np.float32)
        self.C = int(nf.shape[0])
        total = int(nf.sum())
        if rp.shape != (total, 3) or lq.shape != (total, skel.J, 4) or f.shape != (self.C,):
            raise ValueError("clip arrays have inconsistent shapes")
        self.h = C.c_void_p()
        _check(L.im_load_clips(skel.h, self.C, _ptr(nf), _ptr(f), _ptr(rp), _ptr(lq), C.byref(self.h)),
               "im_load_clips")

    def set_cyclic(self, flags=None):
        """Marks clips as played in a loop (one byte per clip; None clears all)."""
        f = None if flags is None else _np(flags, np.uint8)
        if f is not None and f.shape != (self.C,):
            raise ValueError("one flag per clip")
        _check(load().im_clips_set_cyclic(self.h, _ptr(f)), "im_clips_set_cyclic")

    def __del__(self):
        if getattr(self, "h", None) and _lib is not None:
            _lib.im_destroy_clips(self.h)
            self.h = None


def make_env_config(n_envs: int, dt: float, seed: int, reward: dict, h_min: float, ld_obs: int,
                    r_min: float = -np.inf, env_id_base: int = 0, write_back_reset: bool = False,
                    grace_steps: int = 0, reset_noise_std: float = 0.0) -> EnvConfig:
    rc = RewardConfig(mode=int(reward["mode"]), h_min=np.float32(h_min), r_min=np.float32(r_min))
    for k in range(N_TERMS):
        rc.a[k] = reward["a"][k]
        rc.w[k] = reward["w"][k]
    return EnvConfig(n_envs=int(n_envs), env_id_base=int(env_id_base), dt=np.float32(dt), seed=int(seed),
                     reward=rc, ld_obs=int(ld_obs), write_back_reset=int(write_back_reset),
                     grace_steps=int(grace_steps), reset_noise_std=np.float32(reset_noise_std))


def padded_ld(D: int, multiple: int = 64) -> int:
    """Row stride that keeps rows 16-byte aligned and a whole number of GEMM K tiles."""
    return (D + multiple - 1) // multiple * multiple


class Env:
    """Per-env state plus the step calls; all tensors are torch CUDA tensors owned by the caller."""

    def __init__(self, skel: Skeleton, clips: Clips, cfg: EnvConfig, stream=None):
        import torch
        L = load()
        self.skel, self.clips, self.cfg = skel, clips, cfg
        self.n, self.J, self.D, self.ld_obs = cfg.n_envs, skel.J, 24 * skel.J + 1, cfg.ld_obs
        self.stream = stream if stream is not None else torch.cuda.current_stream()
        self.n_bins = 0
        self.h = C.c_void_p()
        _check(L.im_env_create(skel.h, clips.h, C.byref(cfg), C.c_void_p(self.stream.cuda_stream), C.byref(self.h)),
               "im_env_create")

    def new_obs(self):
        import torch
        return torch.empty((self.n, self.ld_obs), dtype=torch.float32, device="cuda")

    def reset_all(self, obs_out, step: int = 0):
        _check(load().im_env_reset_all(self.h, step, _ptr(obs_out)), "im_env_reset_all")

    def step(self, step: int, sim, obs_out, reward_out, flags_out, terms_out=None):
        """sim: CUDA fp32 tensor [13J, stride>=n] (pos, quat, linvel, angvel rows)."""
        J = self.J
        stride = sim.stride(0)
        base = sim.data_ptr()
        bs = BodyState(base, base + 3 * J * stride * 4, base + 7 * J * stride * 4, base + 10 * J * stride * 4, stride)
        _check(load().im_env_step(self.h, step, C.byref(bs), _ptr(obs_out), _ptr(reward_out), _ptr(flags_out),
                                  _ptr(terms_out)), "im_env_step")

    def step_aos(self, step: int, pos, quat, linvel, angvel, obs_out, reward_out, flags_out, terms_out=None):
        """One step on simulator-native arrays: CUDA float32 tensors (or views) indexed [env, body, component];
        any strides along env and body, components contiguous."""
        def arr(t, comps):
            if t.dim() != 3 or t.shape[0] != self.n or t.shape[1] != self.J or t.shape[2] != comps or t.stride(2) != 1:
                raise ValueError("expected a [%d, %d, %d] view with contiguous components" % (self.n, self.J, comps))
            return AosArray(t.data_ptr(), t.stride(0), t.stride(1))
        sim = BodyStateAos(arr(pos, 3), arr(quat, 4), arr(linvel, 3), arr(angvel, 3))
        _check(load().im_env_step_aos(self.h, step, C.byref(sim), _ptr(obs_out), _ptr(reward_out), _ptr(flags_out),
                                      _ptr(terms_out)), "im_env_step_aos")

    def get_state(self):
        import torch
        c = torch.empty(self.n, dtype=torch.int32, device="cuda")
        t = torch.empty(self.n, dtype=torch.float32, device="cuda")
        l = torch.empty(self.n, dtype=torch.int32, device="cuda")
        with torch.cuda.stream(self.stream):
            _check(load().im_env_get_state(self.h, _ptr(c), _ptr(t), _ptr(l)), "im_env_get_state")
        self.stream.synchronize()
        return c, t, l

    def set_aos_staging(self, on: bool = True):
        """step_aos through a library-owned [13J][N] staging buffer (faster, allocated here) instead of in place."""
        _check(load().im_env_set_aos_staging(self.h, int(on)), "im_env_set_aos_staging")

    def get_cycles(self):
        """Cycles completed by each env on a looped clip (int32 CUDA tensor)."""
        import torch
        c = torch.empty(self.n, dtype=torch.int32, device="cuda")
        with torch.cuda.stream(self.stream):
            _check(load().im_env_get_cycles(self.h, _ptr(c)), "im_env_get_cycles")
        self.stream.synchronize()
        return c

    def set_cycles(self, cycle):
        _check(load().im_env_set_cycles(self.h, _ptr(cycle)), "im_env_set_cycles")
        self.stream.synchronize()

    def set_state(self, clip_id=None, t=None, ep_len=None):
        _check(load().im_env_set_state(self.h, _ptr(clip_id), _ptr(t), _ptr(ep_len)), "im_env_set_state")
        self.stream.synchronize()

    def set_reset_bins(self, n_bins: int, weights=None):
        """Adaptive episode initialisation: weights [C, n_bins] over (clip, phase bin); 0 bins: uniform."""
        w = None if weights is None else _np(weights, np.float32)
        if w is not None and w.shape != (self.clips.C, n_bins):
            raise ValueError("weights must be [n_clips, n_bins]")
        _check(load().im_env_set_reset_bins(self.h, int(n_bins), _ptr(w)), "im_env_set_reset_bins")
        self.n_bins = int(n_bins)

    def adapt_reset_bins(self, floor_weight: float, clear: bool = True):
        """Adaptive episode initialisation on the device: bin weights = failure counts + floor_weight."""
        _check(load().im_env_adapt_reset_bins(self.h, float(floor_weight), int(clear)), "im_env_adapt_reset_bins")

    def set_obs_extension(self, n_future: int = 1, prev_action=None):
        """Extended observation: end-effector targets of reference frames 2 .. n_future and the previous action
        (a float32 CUDA tensor [n, A] that later steps read; kept alive here).  Returns the observation width."""
        if prev_action is not None and (prev_action.dim() != 2 or prev_action.shape[0] < self.n or prev_action.stride(1) != 1):
            raise ValueError("prev_action must be a [n, A] tensor with contiguous rows")
        A = 0 if prev_action is None else prev_action.shape[1]
        _check(load().im_env_set_obs_extension(self.h, int(n_future), A, _ptr(prev_action) if A else None,
                                               prev_action.stride(0) if A else 0), "im_env_set_obs_extension")
        self._prev_action = prev_action
        self.n_future = int(n_future)
        self.D = 24 * self.J + 1 + (int(n_future) - 1) * 9 * self.skel.n_ee + A
        return self.D

    def set_summary(self, acc=None):
        """Attaches (None: detaches) a 4-element int64 CUDA tensor every later step adds to: fixed-point reward sum
        (2^-40 units), terminated count, truncated count, summed lengths of the episodes that ended."""
        import torch
        if acc is not None and (acc.dtype != torch.int64 or acc.numel() != 4 or not acc.is_cuda or not acc.is_contiguous()):
            raise ValueError("acc must be a contiguous int64 CUDA tensor of 4 elements")
        _check(load().im_env_set_summary(self.h, _ptr(acc)), "im_env_set_summary")
        self._summary = acc

    def reset_stats(self, clear: bool = False):
        """(starts, failures) per (clip, phase bin) as CUDA int32 tensors [C, n_bins] (uint32 counts)."""
        import torch
        with torch.cuda.stream(self.stream):
            starts = torch.empty((self.clips.C, self.n_bins), dtype=torch.int32, device="cuda")
            failures = torch.empty_like(starts)
            _check(load().im_env_get_reset_stats(self.h, _ptr(starts), _ptr(failures), int(clear)),
                   "im_env_get_reset_stats")
        self.stream.synchronize()
        return starts, failures

    def attach_policy(self, policy):
        """The env also writes bf16 observation rows into the policy's input staging buffer."""
        _check(load().im_env_attach_policy(self.h, None if policy is None else policy.h), "im_env_attach_policy")

    def reset_all_host(self, step: int = 0):
        _check(load().im_env_reset_all_host(self.h, step), "im_env_reset_all_host")

    def device_status(self) -> int:
        out = C.c_uint32(0)
        _check(load().im_poll_device_status(self.h, None, C.byref(out)), "im_poll_device_status")
        return int(out.value)

    def __del__(self):
        if getattr(self, "h", None) and _lib is not None:
            _lib.im_env_destroy(self.h)
            self.h = None


class Policy:
    def __init__(self, dims: Sequence[int], W, b, dtype: str, sigma: float, seed: int, max_batch: int,
                 env_id_base: int = 0, impl: int = 0, stream=None):
        """W[l]: numpy [dims[l+1], dims[l]], float32 (dtype 'f32') or uint16 bf16 bit patterns ('bf16')."""
        import torch
        L = load()
        nl = len(dims) - 1
        cfg = PolicyConfig(n_layers=nl, dtype=1 if dtype == "bf16" else 0, sigma=np.float32(sigma), seed=int(seed),
                           env_id_base=int(env_id_base), max_batch=int(max_batch), impl=int(impl))
        for i, d in enumerate(dims):
            cfg.dims[i] = int(d)
        wt = np.uint16 if dtype == "bf16" else np.float32
        Wc = [_np(w, wt) for w in W]
        bc = [_np(x, np.float32) for x in b]
        for l in range(nl):
            if Wc[l].shape != (dims[l + 1], dims[l]) or bc[l].shape != (dims[l + 1],):
                raise ValueError("layer %d has the wrong shape" % l)
        Wp = (C.c_void_p * nl)(*[w.ctypes.data for w in Wc])
        bp = (C.c_void_p * nl)(*[x.ctypes.data for x in bc])
        self.dims, self.A, self.max_batch = tuple(dims), int(dims[-1]), int(max_batch)
        self.stream = stream if stream is not None else torch.cuda.current_stream()
        self.h = C.c_void_p()
        _check(L.im_load_policy(C.byref(cfg), C.cast(Wp, C.c_void_p), C.cast(bp, C.c_void_p),
                                C.c_void_p(self.stream.cuda_stream), C.byref(self.h)), "im_load_policy")

    def forward(self, step: int, obs, mean_out, action_out, logp_out=None, n: Optional[int] = None):
        n = obs.shape[0] if n is None else n
        _check(load().im_policy_forward(self.h, step, n, _ptr(obs), obs.stride(0), _ptr(mean_out),
                                        _ptr(action_out), _ptr(logp_out)), "im_policy_forward")

    def forward_staged(self, step: int, n: int, mean_out, action_out, logp_out=None):
        """Forward on the bf16 rows an attached env left in the input staging buffer."""
        _check(load().im_policy_forward_staged(self.h, step, n, _ptr(mean_out), _ptr(action_out), _ptr(logp_out)),
               "im_policy_forward_staged")

    def set_log_std(self, log_std):
        """Per-dimension standard deviation exp(log_std): CUDA float32 tensor [A], or None for the scalar sigma."""
        if log_std is not None and (tuple(log_std.shape) != (self.A,) or not log_std.is_contiguous()):
            raise ValueError("log_std must be a contiguous [A] tensor")
        _check(load().im_policy_set_log_std(self.h, _ptr(log_std)), "im_policy_set_log_std")

    def layer_buffers(self, layer: int):
        """(weight pointer, row stride in elements, bias pointer) of a layer on the device."""
        w, b, ld = C.c_void_p(), C.c_void_p(), C.c_int32()
        _check(load().im_policy_layer_buffers(self.h, layer, C.byref(w), C.byref(ld), C.byref(b)),
               "im_policy_layer_buffers")
        return w.value, int(ld.value), b.value

    def value_forward(self, obs, value_out, n: Optional[int] = None):
        """This network read as a critic: writes only its outputs ([n, dims[-1]]), draws no noise."""
        n = obs.shape[0] if n is None else n
        _check(load().im_value_forward(self.h, n, _ptr(obs), obs.stride(0), _ptr(value_out)), "im_value_forward")

    def value_forward_staged(self, n: int, value_out, src: Optional["Policy"] = None):
        """Critic forward on the bf16 rows an env attached to `src` (default: this policy) has staged."""
        _check(load().im_value_forward_staged(self.h, src.h if src is not None else None, n, _ptr(value_out)),
               "im_value_forward_staged")

    def device_status(self) -> int:
        out = C.c_uint32(0)
        _check(load().im_poll_device_status(None, self.h, C.byref(out)), "im_poll_device_status")
        return int(out.value)

    def __del__(self):
        if getattr(self, "h", None) and _lib is not None:
            _lib.im_destroy_policy(self.h)
            self.h = None


def step_host(env: Env, policy: Policy, step: int, sim_host, action_host, reward_host, flags_host):
    """One whole step from host buffers (numpy arrays or pinned CPU torch tensors)."""
    _check(load().im_step_host(env.h, policy.h, step, _ptr(sim_host), _ptr(action_host), _ptr(reward_host),
                               _ptr(flags_host)), "im_step_host")


def gae(reward, value, flags, advantage, returns, gamma: float, lam: float, bootstrap_truncated: bool = True,
        stream=None):
    """Generalised advantage estimation over a rollout.  CUDA tensors, time-major: reward, flags (uint8),
    advantage, returns [T, N] and value [T + 1, N], all with the same row stride."""
    import torch
    T, N = reward.shape
    ld = reward.stride(0) if T > 1 else max(N, value.stride(0))
    for a, rows in ((value, T + 1), (flags, T), (advantage, T), (returns, T)):
        if a.shape != (rows, N) or (rows > 1 and a.stride(0) != ld) or a.stride(1) != 1:
            raise ValueError("rollout arrays must be [T, N] (value [T + 1, N]) with one common row stride")
    cfg = GaeConfig(np.float32(gamma), np.float32(lam), int(bool(bootstrap_truncated)))
    st = stream if stream is not None else torch.cuda.current_stream()
    _check(load().im_gae(C.byref(cfg), T, N, ld, _ptr(reward), _ptr(value), _ptr(flags), _ptr(advantage),
                         _ptr(returns), C.c_void_p(st.cuda_stream)), "im_gae")


def ppo_workspace():
    """Scratch tensor for moments() and ppo_loss()."""
    import torch
    return torch.empty(load().im_ppo_workspace_bytes() // 8, dtype=torch.float64, device="cuda")


def moments(x, out2, workspace, stream=None):
    """out2 <- (mean, 1 / (std + 1e-8)) of the CUDA float32 tensor x (std with the n - 1 divisor)."""
    import torch
    st = stream if stream is not None else torch.cuda.current_stream()
    if not x.is_contiguous():
        raise ValueError("x must be contiguous")
    _check(load().im_moments(_ptr(x), x.numel(), _ptr(out2), _ptr(workspace), C.c_void_p(st.cuda_stream)), "im_moments")


def ppo_loss(batch: dict, d_mean, d_log_std, d_value, summary, workspace, clip: float, value_coef: float,
             entropy_coef: float, clip_value_loss: bool, adv_moments=None, stream=None):
    """PPO minibatch loss and output gradients.  batch: contiguous CUDA float32 tensors mean, action,
    mean_old [M, A]; log_std, log_std_old [A]; logp_old, advantage, value, value_old, returns [M]."""
    import torch
    M, A = batch["mean"].shape
    for k, v in batch.items():
        if not v.is_contiguous() or v.dtype != torch.float32:
            raise ValueError("batch[%r] must be a contiguous float32 tensor" % k)
    b = PpoBatch(**{k: batch[k].data_ptr() for k in ("mean", "log_std", "action", "logp_old", "mean_old",
                                                      "log_std_old", "advantage", "value", "returns")})
    b.value_old = batch["value_old"].data_ptr() if batch.get("value_old") is not None else None
    b.adv_moments = adv_moments.data_ptr() if adv_moments is not None else None
    cfg = PpoConfig(np.float32(clip), np.float32(value_coef), np.float32(entropy_coef), int(bool(clip_value_loss)))
    st = stream if stream is not None else torch.cuda.current_stream()
    _check(load().im_ppo_loss(C.byref(cfg), M, A, C.byref(b), _ptr(d_mean), _ptr(d_log_std), _ptr(d_value),
                              _ptr(summary), _ptr(workspace), C.c_void_p(st.cuda_stream)), "im_ppo_loss")


def adam_step(param, grad, m, v, lr, t: int, beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8,
              grad_scale=None, bf16_out_ptr: Optional[int] = None, cols: int = 0, ld_bf16: int = 0, stream=None):
    """Fused Adam step on contiguous CUDA float32 tensors; lr (and grad_scale) are 1-element CUDA tensors."""
    import torch
    for a in (param, grad, m, v):
        if not a.is_contiguous() or a.dtype != torch.float32 or a.numel() != param.numel():
            raise ValueError("param, grad, m, v must be contiguous float32 tensors of one size")
    cfg = AdamConfig(np.float32(beta1), np.float32(beta2), np.float32(eps))
    st = stream if stream is not None else torch.cuda.current_stream()
    _check(load().im_adam_step(C.byref(cfg), int(t), param.numel(), _ptr(param), _ptr(grad), _ptr(m), _ptr(v), _ptr(lr),
                               _ptr(grad_scale), C.c_void_p(bf16_out_ptr) if bf16_out_ptr else None, int(cols),
                               int(ld_bf16), C.c_void_p(st.cuda_stream)), "im_adam_step")


def grad_scale(grads, max_norm: float, scale_out, workspace, stream=None):
    """scale_out[0:2] <- (min(1, max_norm / (global L2 norm + 1e-6)), norm) over a list of CUDA float32 tensors."""
    import torch
    ptrs = (C.c_void_p * len(grads))(*[g.data_ptr() for g in grads])
    sizes = np.asarray([g.numel() for g in grads], np.int64)
    st = stream if stream is not None else torch.cuda.current_stream()
    _check(load().im_grad_scale(len(grads), C.cast(ptrs, C.c_void_p), _ptr(sizes), C.c_float(max_norm), _ptr(scale_out),
                                _ptr(workspace), C.c_void_p(st.cuda_stream)), "im_grad_scale")


def adaptive_lr(lr, kl, kl_target: float, lr_min: float = 1e-5, lr_max: float = 1e-2, stream=None):
    """lr (1-element CUDA tensor) follows the mean KL (1-element CUDA tensor or view) against kl_target."""
    import torch
    st = stream if stream is not None else torch.cuda.current_stream()
    _check(load().im_adaptive_lr(_ptr(lr), _ptr(kl), C.c_float(kl_target), C.c_float(lr_min), C.c_float(lr_max),
                                 C.c_void_p(st.cuda_stream)), "im_adaptive_lr")


# ---- backward-pass building blocks: 2-D CUDA tensors, bf16 as torch.bfloat16, row stride = stride(0)
def _st(stream):
    import torch
    return C.c_void_p((stream if stream is not None else torch.cuda.current_stream()).cuda_stream)


def gemm_bf16(A, B, Cout, bias, relu: bool, status, stream=None):
    """Cout[M, N] (bf16) = act(A[M, K] @ B[N, K].T + bias)."""
    M, K = A.shape
    N = B.shape[0]
    _check(load().im_gemm_bf16(_ptr(A), A.stride(0), _ptr(B), B.stride(0), _ptr(Cout), Cout.stride(0), M, N, K,
                               _ptr(bias), int(relu), _ptr(status), _st(stream)), "im_gemm_bf16")


def gemm_bf16_tn(A, Bm, Cout, slices: int, c_pitch: int, status, stream=None):
    """Cout (bf16, [slices * c_pitch, No]): slice s holds A[rows of s].T @ Bm[rows of s]; A [R, Mo], Bm [R, No]."""
    R, Mo = A.shape
    No = Bm.shape[1]
    _check(load().im_gemm_bf16_tn(_ptr(A), A.stride(0), _ptr(Bm), Bm.stride(0), _ptr(Cout), Cout.stride(0), R, Mo, No,
                                  slices, c_pitch, _ptr(status), _st(stream)), "im_gemm_bf16_tn")


def sum_slices_bf16_to_f32(x, slices: int, rows: int, cols: int, out, stream=None):
    """out (dense float32 [rows, cols]) = sum of the `slices` row blocks of x ([slices * R, ld] bf16, R = x.shape[0] // slices)."""
    R = x.shape[0] // slices
    _check(load().im_sum_slices_bf16_to_f32(_ptr(x), R * x.stride(0), x.stride(0), slices, rows, cols, _ptr(out), _st(stream)),
           "im_sum_slices_bf16_to_f32")


def gemm_bf16_f32out(A, B, Cout, bias, status, stream=None):
    """Cout[M, N] (float32, dense, N <= 80) = A[M, K] @ B[:N, K].T + bias; B and bias padded to 16 rows."""
    M, K = A.shape
    N = Cout.shape[1]
    _check(load().im_gemm_bf16_f32out(_ptr(A), A.stride(0), _ptr(B), B.stride(0), _ptr(Cout), M, N, K, _ptr(bias),
                                      _ptr(status), _st(stream)), "im_gemm_bf16_f32out")


def transpose_bf16(x, out, stream=None):
    _check(load().im_transpose_bf16(_ptr(x), x.stride(0), x.shape[0], x.shape[1], _ptr(out), out.stride(0), _st(stream)),
           "im_transpose_bf16")


def f32_to_bf16_padded(x, out, stream=None):
    _check(load().im_f32_to_bf16_padded(_ptr(x), x.stride(0), x.shape[0], x.shape[1], _ptr(out), out.stride(0),
                                        _st(stream)), "im_f32_to_bf16_padded")


def f32_to_bf16_padded_ptr(x, out_ptr: int, ld_out: int, stream=None):
    """Like f32_to_bf16_padded, into a raw device pointer (a policy's weight matrix from Policy.layer_buffers)."""
    _check(load().im_f32_to_bf16_padded(_ptr(x), x.stride(0), x.shape[0], x.shape[1], C.c_void_p(out_ptr), int(ld_out),
                                        _st(stream)), "im_f32_to_bf16_padded")


def gemm_bf16_dgrad(dZ, Wt, dH, H, colsum_partial, status, stream=None):
    """dH [M, N] = (H > 0) * (dZ [M, K] @ Wt [N, K]^T) as bf16, and the fp32 column sums of dH per 32-row block into
    colsum_partial [M / 32, >= N] float32.  H and colsum_partial may be None."""
    M, K = dZ.shape
    N = Wt.shape[0]
    _check(load().im_gemm_bf16_dgrad(_ptr(dZ), dZ.stride(0), _ptr(Wt), Wt.stride(0), _ptr(dH), dH.stride(0), M, N, K,
                                     _ptr(H) if H is not None else None, H.stride(0) if H is not None else 0,
                                     _ptr(colsum_partial) if colsum_partial is not None else None,
                                     colsum_partial.stride(0) if colsum_partial is not None else 0, _ptr(status),
                                     _st(stream)), "im_gemm_bf16_dgrad")


def gather_rows(x, idx, out, status, stream=None):
    """out[i] = x[idx[i]] for a float32 [R, cols] source (1-D sources are taken as one column); out float32 with
    x's width, or bfloat16 [M, ld] zero padded.  idx: int32 CUDA tensor."""
    import torch
    x2 = x if x.dim() == 2 else x.view(-1, 1)
    o2 = out if out.dim() == 2 else out.view(-1, 1)
    _check(load().im_gather_rows_f32(_ptr(x2), x2.stride(0), _ptr(idx), x2.shape[0], idx.numel(), x2.shape[1], _ptr(o2),
                                     o2.stride(0), int(out.dtype == torch.bfloat16), _ptr(status), _st(stream)),
           "im_gather_rows_f32")


def copy_f32_ptr(dst_ptr: int, src, stream=None):
    _check(load().im_copy_f32(C.c_void_p(dst_ptr), _ptr(src), src.numel(), _st(stream)), "im_copy_f32")


def colsum(x, out, workspace, stream=None):
    """out[c] = sum over rows of the float32 matrix x."""
    _check(load().im_colsum_f32(_ptr(x), x.stride(0), x.shape[0], x.shape[1], _ptr(out), _ptr(workspace),
                                workspace.numel() * workspace.element_size(), _st(stream)), "im_colsum_f32")


class _DeviceArray:
    """A device array owned by a library handle, described the way torch.as_tensor understands."""

    def __init__(self, ptr: int, shape, typestr: str, strides=None):
        self.__cuda_array_interface__ = dict(shape=tuple(shape), typestr=typestr, data=(int(ptr), False), version=3,
                                             strides=strides)


def device_tensor(ptr: int, shape, dtype: str, row_stride: Optional[int] = None):
    """torch view (no copy) of `shape` elements at device address ptr; dtype 'f32', 'bf16' or 'u32';
    row_stride in elements for 2-D arrays whose rows are padded.  The owner of the memory must outlive the view."""
    import torch
    typestr, esz = {"f32": ("<f4", 4), "bf16": ("<i2", 2), "u32": ("<i4", 4)}[dtype]
    strides = None
    if len(shape) == 2 and row_stride is not None and row_stride != shape[1]:
        strides = (row_stride * esz, esz)
    t = torch.as_tensor(_DeviceArray(ptr, shape, typestr, strides), device="cuda")
    return t.view(torch.bfloat16) if dtype == "bf16" else t


NOALLOC_MAX_BATCH = 1024
NOALLOC_MAX_WIDTH = 1024
DEBUG_ANGLE_SQ, DEBUG_SLERP = 0, 1


def debug_set_wait(limit_ns: int = 2_000_000_000, skip_loads: bool = False):
    """Limit of the kernels' bounded waits on the current device; skip_loads makes the copy-issuing threads idle."""
    _check(load().im_debug_set_wait(int(limit_ns), int(skip_loads)), "im_debug_set_wait")


def debug_math(op: int, inp):
    """The env kernel's angle / slerp device functions on rows of `inp` (float32 CUDA tensor, [n, 4] or [n, 8])."""
    import torch
    assert inp.is_cuda and inp.dtype == torch.float32 and inp.is_contiguous()
    n = inp.shape[0]
    out = torch.empty(n if op == DEBUG_ANGLE_SQ else (n, 7), device=inp.device)
    _check(load().im_debug_math(op, n, inp.data_ptr(), out.data_ptr(), torch.cuda.current_stream().cuda_stream), "im_debug_math")
    return out


def policy_forward_noalloc(dims: Sequence[int], W_dev, b_dev, sigma: float, seed: int, step: int, obs,
                           mean_out, action_out, logp_out=None, env_id_base: int = 0, n: Optional[int] = None,
                           stream=None):
    """fp32 policy forward that allocates nothing: for callers that cannot call cudaMalloc when they
    need an action (latency-bound control loops, processes with a fixed memory budget).  W_dev and
    b_dev are lists of CUDA float32 tensors the caller owns; the hidden activations live in a fixed
    8 MiB array inside the library, shared by all calls on the device, so calls must not overlap on
    the GPU.  At most NOALLOC_MAX_BATCH rows and hidden widths up to NOALLOC_MAX_WIDTH."""
    import torch
    L = load()
    nl = len(dims) - 1
    d = np.asarray(dims, np.int32)
    Wp = (C.c_void_p * nl)(*[w.data_ptr() for w in W_dev])
    bp = (C.c_void_p * nl)(*[x.data_ptr() for x in b_dev])
    st = stream if stream is not None else torch.cuda.current_stream()
    n = obs.shape[0] if n is None else n
    _check(L.im_policy_forward_noalloc(nl, _ptr(d), C.cast(Wp, C.c_void_p), C.cast(bp, C.c_void_p),
                                       C.c_float(sigma), int(seed), int(env_id_base), int(step), int(n),
                                       _ptr(obs), obs.stride(0), _ptr(mean_out), _ptr(action_out),
                                       _ptr(logp_out), C.c_void_p(st.cuda_stream)), "im_policy_forward_noalloc")
