"""Python face of the update phase (`im_trainer_*`, `im_ppo_*` of the C ABI): argument marshalling only.
The layer loop, the buffer plan, the row-slice choice of the dW products, the optimiser sequencing and the
minibatch loop over a rollout all live in the library (csrc/trainer.cu); the attributes below are torch views
of arrays the library handles own.
"""
from __future__ import annotations

import ctypes as C
from typing import List, Optional, Sequence

import numpy as np
import torch

from . import binding as B

# im_trainer_tensor / im_ppo_updater_tensor selectors (include/im.h)
_W, _B, _WB, _WBT, _MW, _VW, _MB, _VB, _DW, _DB, _H, _OUT, _STATUS = range(13)
_LOG_STD, _LOG_STD_OLD, _M_LS, _V_LS, _LR, _SCALE, _SUMMARY = range(7)
_DTYPES = {0: "f32", 1: "bf16", 2: "u32"}


def dw_slices(Np: int, Kp: int, M: int, max_split: int = 64, any_rows: bool = False) -> int:
    """Row slices the library takes for the dW product of a layer with Np x Kp padded weights on M rows."""
    return int(B.load().im_trainer_dw_slices(Np, Kp, M, max_split, int(any_rows)))


class MlpTrainer:
    """One MLP in training form (handle of im_trainer_create) for minibatches of up to max_rows rows."""

    def __init__(self, dims: Sequence[int], W: List[np.ndarray], b: List[np.ndarray], max_rows: int, stream=None):
        self.dims = tuple(int(d) for d in dims)
        self.nl = len(self.dims) - 1
        self.Mb = int(max_rows)
        self.stream = stream if stream is not None else torch.cuda.current_stream()
        Wc = [np.ascontiguousarray(w, np.float32) for w in W]
        bc = [np.ascontiguousarray(x, np.float32) for x in b]
        for l in range(self.nl):
            if Wc[l].shape != (self.dims[l + 1], self.dims[l]) or bc[l].shape != (self.dims[l + 1],):
                raise ValueError("layer %d: weight / bias shape" % l)
        Wp = (C.c_void_p * self.nl)(*[w.ctypes.data for w in Wc])
        bp = (C.c_void_p * self.nl)(*[x.ctypes.data for x in bc])
        d = np.asarray(self.dims, np.int32)
        h = C.c_void_p()
        B._check(B.load().im_trainer_create(self.nl, d.ctypes.data, C.cast(Wp, C.c_void_p), C.cast(bp, C.c_void_p), self.Mb,
                                            C.c_void_p(self.stream.cuda_stream), C.byref(h)), "im_trainer_create")
        self.h = h
        per_layer = lambda which: [self._tensor(which, l) for l in range(self.nl)]
        self.W, self.Wb, self.WbT = per_layer(_W), per_layer(_WB), per_layer(_WBT)
        self.mW, self.vW, self.mb, self.vb = per_layer(_MW), per_layer(_VW), per_layer(_MB), per_layer(_VB)
        self.dW, self.db = per_layer(_DW), per_layer(_DB)
        self.b = per_layer(_B)                       # views of the dims[l+1] biases
        self.H0 = self._tensor(_H, 0)
        self.out = self._tensor(_OUT, 0)
        self.status = self._tensor(_STATUS, 0)

    def _tensor(self, which: int, layer: int) -> torch.Tensor:
        ptr, rows, cols, ld, dt = C.c_void_p(), C.c_int64(), C.c_int64(), C.c_int64(), C.c_int32()
        B._check(B.load().im_trainer_tensor(self.h, which, layer, C.byref(ptr), C.byref(rows), C.byref(cols), C.byref(ld),
                                            C.byref(dt)), "im_trainer_tensor")
        if which in (_B, _MB, _VB, _DB, _STATUS):                  # vectors
            return B.device_tensor(ptr.value, (cols.value,), _DTYPES[dt.value])
        return B.device_tensor(ptr.value, (rows.value, cols.value), _DTYPES[dt.value], ld.value)

    def __del__(self):
        if getattr(self, "h", None) and B is not None:
            try:
                torch.cuda.synchronize()
                B.load().im_trainer_destroy(self.h)
            except Exception:
                pass
            self.h = None

    def input_rows(self, M: int) -> torch.Tensor:
        """bf16 view [M, padded dims[0]] the caller fills with the (zero-padded) observations."""
        return self.H0[:M]

    def forward(self, M: int) -> torch.Tensor:
        """Runs the net on input_rows(M); returns the fp32 outputs [M, dims[-1]] (a view)."""
        B._check(B.load().im_trainer_forward(self.h, M), "im_trainer_forward")
        return self.out[:M]

    def backward(self, d_out: torch.Tensor, M: int):
        """d_out: float32 [M, dims[-1]] = dL/d(outputs) of the forward just run on M rows (M % 64 == 0).
        Fills dW[l] (float32 [N, K]) and db[l] (float32 [N])."""
        if d_out.dtype != torch.float32 or not d_out.is_contiguous() or d_out.numel() != M * self.dims[-1]:
            raise ValueError("d_out must be a contiguous float32 [M, dims[-1]] tensor")
        B._check(B.load().im_trainer_backward(self.h, B._ptr(d_out), M), "im_trainer_backward")

    def grads(self) -> List[torch.Tensor]:
        return self.dW + self.db

    def step(self, lr: torch.Tensor, grad_scale: Optional[torch.Tensor] = None, beta1=0.9, beta2=0.999, eps=1e-8):
        """Adam step on every tensor; the bf16 working copies (and their transposes) follow."""
        cfg = B.AdamConfig(beta1, beta2, eps)
        B._check(B.load().im_trainer_step(self.h, C.byref(cfg), B._ptr(lr), B._ptr(grad_scale) if grad_scale is not None else None),
                 "im_trainer_step")

    def set_step_count(self, t: int):
        B._check(B.load().im_trainer_set_step_count(self.h, t), "im_trainer_set_step_count")

    def push_to_policy(self, policy: B.Policy):
        """Writes the current weights into a loaded policy of the same shape and stream."""
        B._check(B.load().im_trainer_push_to_policy(self.h, policy.h), "im_trainer_push_to_policy")

    def device_status(self) -> int:
        return int(self.status.item())


class PpoUpdater:
    """One actor, one critic and the learnable log-std (handle of im_ppo_updater_create): `update` is one PPO
    minibatch update, `update_from_storage` the whole update phase over a collected rollout."""

    def __init__(self, actor: MlpTrainer, critic: MlpTrainer, log_std: torch.Tensor, lr: float, clip: float = 0.2,
                 value_coef: float = 2.0, entropy_coef: float = 0.0, clip_value_loss: bool = True,
                 max_grad_norm: float = 1.0, kl_target: float = 0.008, normalize_advantage: bool = True,
                 lr_min: float = 1e-5, lr_max: float = 1e-2):
        self.actor, self.critic, self.stream = actor, critic, actor.stream
        self.A, self.Mb = actor.dims[-1], actor.Mb
        ls = np.ascontiguousarray(log_std.detach().cpu().numpy(), np.float32)
        if ls.shape != (self.A,):
            raise ValueError("log_std must have one entry per action dimension")
        cfg = B.PpoUpdateConfig(lr, clip, value_coef, entropy_coef, int(clip_value_loss), max_grad_norm, kl_target, lr_min,
                                lr_max, int(normalize_advantage), B.AdamConfig(0.9, 0.999, 1e-8))
        h = C.c_void_p()
        B._check(B.load().im_ppo_updater_create(actor.h, critic.h, ls.ctypes.data, C.byref(cfg), C.byref(h)),
                 "im_ppo_updater_create")
        self.h = h
        t = lambda which: self._tensor(which)
        self.log_std, self.log_std_old, self.m_ls, self.v_ls = t(_LOG_STD), t(_LOG_STD_OLD), t(_M_LS), t(_V_LS)
        self.lr, self.scale, self.summary = t(_LR), t(_SCALE), t(_SUMMARY)

    def _tensor(self, which: int) -> torch.Tensor:
        ptr, n = C.c_void_p(), C.c_int64()
        B._check(B.load().im_ppo_updater_tensor(self.h, which, C.byref(ptr), C.byref(n)), "im_ppo_updater_tensor")
        return B.device_tensor(ptr.value, (n.value,), "f32")

    def __del__(self):
        if getattr(self, "h", None) and B is not None:
            try:
                torch.cuda.synchronize()
                B.load().im_ppo_updater_destroy(self.h)
            except Exception:
                pass
            self.h = None

    def set_step_count(self, t: int):
        B._check(B.load().im_ppo_updater_set_step_count(self.h, t), "im_ppo_updater_set_step_count")

    def update(self, M: int, batch: dict):
        """batch: contiguous CUDA float32 tensors action, mean_old [M, A]; logp_old, advantage, value_old,
        returns [M]; optionally log_std_old [A].  The minibatch observations must already sit (bf16, zero
        padded) in actor.input_rows(M) and critic.input_rows(M).  M % 64 == 0."""
        p = lambda k: B._ptr(batch[k]) if batch.get(k) is not None else None
        mb = B.PpoMinibatch(p("action"), p("mean_old"), p("log_std_old"), p("logp_old"), p("advantage"), p("value_old"),
                            p("returns"))
        B._check(B.load().im_ppo_update(self.h, M, C.byref(mb)), "im_ppo_update")


def update_from_storage(upd: PpoUpdater, storage, epochs: int, n_minibatches: int, perm: torch.Tensor = None):
    """The update phase over one collected rollout (im_ppo_update_rollout): `epochs` passes over `n_minibatches`
    blocks of the T * N samples; perm: int32 CUDA tensor [epochs, T * N] for shuffled minibatches.
    Enqueues only; capturable in a CUDA graph together with the rollout."""
    T, N, A = storage.T, storage.N, storage.A
    if not storage.keep_obs:
        raise ValueError("the update reads the stored observations")
    if perm is not None and (perm.dtype != torch.int32 or tuple(perm.shape) != (epochs, T * N) or not perm.is_contiguous()):
        raise ValueError("perm must be a contiguous int32 tensor [epochs, T * N]")
    view = B.RolloutView(T, N, A, storage.ld_obs, B._ptr(storage.obs), B._ptr(storage.action), B._ptr(storage.mean),
                         B._ptr(storage.logp), B._ptr(storage.advantage), B._ptr(storage.returns), B._ptr(storage.value))
    B._check(B.load().im_ppo_update_rollout(upd.h, C.byref(view), epochs, n_minibatches, B._ptr(perm) if perm is not None else None),
             "im_ppo_update_rollout")
