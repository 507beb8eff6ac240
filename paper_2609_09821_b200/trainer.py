"""Training-side sequencing of the C-ABI calls for one MLP (actor or critic): forward that keeps
every layer's activation, backward pass, optimiser step.  Argument marshalling only -- every
arithmetic step runs in the CUDA library:

    forward    hidden layers  im_gemm_bf16 (bias + ReLU fused, bf16 activations kept per layer)
               last layer     im_gemm_bf16_f32out (fp32 outputs)
    backward   dZ_L           im_f32_to_bf16_padded(dL/d output)            db_L  im_colsum_f32
               per layer      im_gemm_bf16_tn -> partial dW per row slice (bf16, operands read in place),
                              im_sum_slices_bf16_to_f32 -> dW
                              im_gemm_bf16_dgrad with W^T -> dZ_{l-1} = (H > 0) * (dZ W) and its 32-row column
                              sums (both in the product's epilogue), im_colsum_f32 of those -> db_{l-1}
    step       im_grad_scale (global norm), im_adam_step per tensor (writes the bf16 weights in place),
               im_transpose_bf16 refreshes W^T

Shapes are padded to what the tensor-core kernels take: widths to multiples of 64 (zero padding, which
the arithmetic leaves zero), batch rows M to a multiple of 64.
"""
from __future__ import annotations

from typing import List, Sequence

import numpy as np
import torch

from . import binding as B


def _pad64(x: int) -> int:
    return (x + 63) // 64 * 64


class MlpTrainer:
    """fp32 master weights + Adam state + bf16 working copies of one MLP, and its buffers for up to max_rows samples."""

    def __init__(self, dims: Sequence[int], W: List[np.ndarray], b: List[np.ndarray], max_rows: int, stream=None):
        if max_rows % 64:
            raise ValueError("max_rows must be a multiple of 64")
        self.dims = tuple(int(d) for d in dims)
        self.nl = len(dims) - 1
        self.Mb = int(max_rows)
        self.stream = stream if stream is not None else torch.cuda.current_stream()
        dev, bf, f32 = "cuda", torch.bfloat16, torch.float32
        self.Kp = [_pad64(d) for d in self.dims[:-1]]
        self.Np = [_pad64(d) for d in self.dims[1:]]
        self.W, self.b, self.Wb, self.WbT = [], [], [], []
        self.mW, self.vW, self.mb, self.vb, self.dW, self.db = [], [], [], [], [], []
        for l in range(self.nl):
            N, K = self.dims[l + 1], self.dims[l]
            w = torch.from_numpy(np.ascontiguousarray(W[l], np.float32)).to(dev)
            self.W.append(w)
            bias = torch.zeros(self.Np[l], dtype=f32, device=dev)          # padded: the GEMM epilogue reads whole tiles
            bias[:N] = torch.from_numpy(np.ascontiguousarray(b[l], np.float32)).to(dev)
            self.b.append(bias)
            wb = torch.zeros((self.Np[l], self.Kp[l]), dtype=bf, device=dev)
            wb[:N, :K] = w.to(bf)
            self.Wb.append(wb)
            self.WbT.append(torch.zeros((self.Kp[l], self.Np[l]), dtype=bf, device=dev))
            self.mW.append(torch.zeros_like(w)); self.vW.append(torch.zeros_like(w))
            self.mb.append(torch.zeros(N, dtype=f32, device=dev)); self.vb.append(torch.zeros(N, dtype=f32, device=dev))
            self.dW.append(torch.zeros_like(w)); self.db.append(torch.zeros(N, dtype=f32, device=dev))
        Mb = self.Mb
        self.H = [torch.zeros((Mb, self.Kp[0]), dtype=bf, device=dev)]
        self.H += [torch.zeros((Mb, self.Np[l]), dtype=bf, device=dev) for l in range(self.nl - 1)]
        self.out = torch.zeros((Mb, self.dims[-1]), dtype=f32, device=dev)
        self.dZ = [torch.zeros((Mb, self.Np[l]), dtype=bf, device=dev) for l in range(self.nl)]
        self.max_split = 64                                                 # most slices of the batch dimension in a dW GEMM
        # partial dW products of one layer: room for the most slices _dw_slices can choose
        need = 0
        for l in range(self.nl):
            npb = (self.Np[l] + 127) // 128 * 128
            s_max = self._dw_slices(l, self.Mb, any_rows=True)     # more rows never favour fewer slices
            need = max(need, s_max * npb * self.Kp[l])
        self.dWs = torch.zeros(need, dtype=bf, device=dev)
        self.zeros = torch.zeros(max(self.Kp + self.Np), dtype=f32, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.colsum_ws = torch.empty(((Mb + 255) // 256) * max(self.Np), dtype=f32, device=dev)
        self.col_partial = torch.empty((Mb // 32, max(self.Np)), dtype=f32, device=dev)   # 32-row column sums of a dH product
        self.t = 0
        with torch.cuda.stream(self.stream):
            for l in range(self.nl):
                B.transpose_bf16(self.Wb[l], self.WbT[l], self.stream)

    def _dw_slices(self, l: int, M: int, any_rows: bool = False) -> int:
        """Row slices of the dW product of layer l on M rows: dW contracts over the batch (a long sum feeding
        few output tiles), so the rows are cut into S slices that run as one launch.  S is the power of two
        (slices of whole 128-row blocks) with the least modelled time: waves of tiles on 148 SMs times rows per
        slice (5 ns per row and wave, measured on the 1024 x 1024 layer), plus the pass that adds the S
        partial products (1 ps per element).  any_rows: ignore the divisibility rule (an upper bound for sizing)."""
        npb = (self.Np[l] + 127) // 128 * 128
        tiles = (npb // 128) * max(1, (self.Kp[l] + 255) // 256)
        best, best_cost, S = 1, None, 1
        while S <= self.max_split and (any_rows or M % (128 * S) == 0):
            cost = 5e-9 * M * -(-tiles * S // 148) / S + 1e-12 * S * npb * self.Kp[l]
            if best_cost is None or cost < best_cost * (1.0 - 1e-9):
                best, best_cost = S, cost
            S *= 2
        return best

    # -- forward ---------------------------------------------------------------
    def input_rows(self, M: int) -> torch.Tensor:
        """bf16 view [M, Kp0] the caller fills with the (zero-padded) observations."""
        return self.H[0][:M]

    def forward(self, M: int) -> torch.Tensor:
        """Runs the net on input_rows(M); returns the fp32 outputs [M, dims[-1]] (a view)."""
        if M < 1 or M > self.Mb:
            raise ValueError("M out of range")
        st = self.stream
        for l in range(self.nl - 1):
            B.gemm_bf16(self.H[l][:M], self.Wb[l], self.H[l + 1][:M], self.b[l], True, self.status, st)
        L = self.nl - 1
        B.gemm_bf16_f32out(self.H[L][:M], self.Wb[L], self.out[:M], self.b[L], self.status, st)
        return self.out[:M]

    # -- backward --------------------------------------------------------------
    def backward(self, d_out: torch.Tensor, M: int):
        """d_out: float32 [M, dims[-1]] = dL/d(outputs) of the forward just run on M rows (M % 64 == 0).
        Fills self.dW[l] (float32 [N, K]) and self.db[l] (float32 [N])."""
        if M % 64 or M < 64 or M > self.Mb:
            raise ValueError("M must be a multiple of 64 within the buffers")
        st = self.stream
        L = self.nl - 1
        B.f32_to_bf16_padded(d_out, self.dZ[L][:M], st)
        B.colsum(d_out, self.db[L], self.colsum_ws, st)
        for l in range(L, -1, -1):
            N, K, Np, Kp = self.dims[l + 1], self.dims[l], self.Np[l], self.Kp[l]
            dZ = self.dZ[l][:M]
            # dW = dZ^T H over S row slices in one launch (im_gemm_bf16_tn reads dZ and H as they are, M/N-major
            # tensor-core operands: no transposed copies); the S partial products are added afterwards
            Npb = (Np + 127) // 128 * 128
            S = self._dw_slices(l, M)
            dWs = self.dWs[:S * Npb * Kp].view(S * Npb, Kp)
            B.gemm_bf16_tn(dZ, self.H[l][:M], dWs, S, Npb, self.zeros, self.status, st)
            B.sum_slices_bf16_to_f32(dWs, S, N, K, self.dW[l], st)
            if l > 0:
                dH = self.dZ[l - 1][:M]                                                       # [M, Kp] = [M, Np of layer l-1]
                # dH = (H > 0) * (dZ W); the GEMM's epilogue applies the ReLU mask and leaves the column sums of
                # every 32-row block, which add up to the bias gradient of the layer below
                part = self.col_partial[:M // 32]
                B.gemm_bf16_dgrad(dZ, self.WbT[l], dH, self.H[l][:M], part, self.zeros, self.status, st)
                B.colsum(part[:, :K], self.db[l - 1], self.colsum_ws, st)

    # -- optimiser -------------------------------------------------------------
    def grads(self) -> List[torch.Tensor]:
        return self.dW + self.db

    def step(self, lr: torch.Tensor, grad_scale: torch.Tensor = None, beta1=0.9, beta2=0.999, eps=1e-8):
        """Adam step on every tensor; the bf16 working copies (and their transposes) follow."""
        self.t += 1
        st = self.stream
        for l in range(self.nl):
            K = self.dims[l]
            B.adam_step(self.W[l], self.dW[l], self.mW[l], self.vW[l], lr, self.t, beta1, beta2, eps, grad_scale,
                        bf16_out_ptr=self.Wb[l].data_ptr(), cols=K, ld_bf16=self.Kp[l], stream=st)
            N = self.dims[l + 1]
            B.adam_step(self.b[l][:N], self.db[l], self.mb[l], self.vb[l], lr, self.t, beta1, beta2, eps, grad_scale,
                        stream=st)
            B.transpose_bf16(self.Wb[l], self.WbT[l], st)

    def push_to_policy(self, policy: B.Policy):
        """Writes the current weights into a loaded tensor-core policy of the same shape (bf16 weight rows
        with the policy's row stride, fp32 biases), so the next rollout acts with the trained network.
        Stream-ordered, no host copy; the policy must use this trainer's stream."""
        if tuple(policy.dims) != self.dims:
            raise ValueError("policy and trainer differ in shape")
        for l in range(self.nl):
            w_ptr, ld, b_ptr = policy.layer_buffers(l)
            B.f32_to_bf16_padded_ptr(self.W[l], w_ptr, ld, self.stream)
            B.copy_f32_ptr(b_ptr, self.b[l][:self.dims[l + 1]], self.stream)

    def device_status(self) -> int:
        return int(self.status.item())


class PpoUpdater:
    """One PPO minibatch update of an actor and a critic (the paper's `update_policy`), every step a
    library kernel and nothing read back on the host: forward of both nets on the minibatch, loss
    and output gradients (im_moments + im_ppo_loss), both backward passes, global-norm clip over all
    gradient tensors, Adam on every tensor, learning rate adapted from the mean KL.
    """

    def __init__(self, actor: MlpTrainer, critic: MlpTrainer, log_std: torch.Tensor, lr: float, clip: float = 0.2,
                 value_coef: float = 2.0, entropy_coef: float = 0.0, clip_value_loss: bool = True,
                 max_grad_norm: float = 1.0, kl_target: float = 0.008, normalize_advantage: bool = True):
        if actor.stream != critic.stream or critic.dims[-1] != 1 or actor.Mb != critic.Mb:
            raise ValueError("actor and critic must share the stream and batch size; the critic has one output")
        self.actor, self.critic, self.stream = actor, critic, actor.stream
        self.A, self.Mb = actor.dims[-1], actor.Mb
        dev, f32 = "cuda", torch.float32
        self.log_std = log_std.detach().clone().to(dev, f32).contiguous()      # learnable parameter [A]
        self.log_std_old = self.log_std.clone()                                # the behaviour policy's, frozen per rollout
        self.m_ls, self.v_ls = torch.zeros_like(self.log_std), torch.zeros_like(self.log_std)
        self.d_log_std = torch.zeros_like(self.log_std)
        self.lr = torch.tensor([lr], dtype=f32, device=dev)
        self.scale = torch.zeros(2, dtype=f32, device=dev)
        self.moments = torch.zeros(2, dtype=f32, device=dev)
        self.summary = torch.zeros(6, dtype=f32, device=dev)
        self.d_mean = torch.zeros((self.Mb, self.A), dtype=f32, device=dev)
        self.d_value = torch.zeros(self.Mb, dtype=f32, device=dev)
        self.ws = B.ppo_workspace()
        self.cfg = dict(clip=clip, value_coef=value_coef, entropy_coef=entropy_coef, clip_value_loss=clip_value_loss)
        self.max_grad_norm, self.kl_target, self.normalize = max_grad_norm, kl_target, normalize_advantage
        self.t = 0

    def update(self, M: int, batch: dict):
        """batch: contiguous CUDA float32 tensors action, mean_old [M, A]; log_std_old [A]; logp_old, advantage,
        value_old, returns [M].  The minibatch observations must already sit (bf16, zero padded) in
        actor.input_rows(M) and critic.input_rows(M).  M % 64 == 0."""
        st = self.stream
        mean = self.actor.forward(M)
        value = self.critic.forward(M)
        b = dict(batch, mean=mean, log_std=self.log_std, value=value.view(M))
        mom = None
        if self.normalize:
            B.moments(batch["advantage"], self.moments, self.ws, st)
            mom = self.moments
        B.ppo_loss(b, self.d_mean[:M], self.d_log_std, self.d_value[:M], self.summary, self.ws,
                   self.cfg["clip"], self.cfg["value_coef"], self.cfg["entropy_coef"], self.cfg["clip_value_loss"],
                   adv_moments=mom, stream=st)
        self.actor.backward(self.d_mean[:M], M)
        self.critic.backward(self.d_value[:M].view(M, 1), M)
        B.grad_scale(self.actor.grads() + self.critic.grads() + [self.d_log_std], self.max_grad_norm, self.scale, self.ws, st)
        self.actor.step(self.lr, self.scale[:1])
        self.critic.step(self.lr, self.scale[:1])
        self.t += 1
        B.adam_step(self.log_std, self.d_log_std, self.m_ls, self.v_ls, self.lr, self.t, grad_scale=self.scale[:1], stream=st)
        B.adaptive_lr(self.lr, self.summary[4:5], self.kl_target, stream=st)


def update_from_storage(upd: PpoUpdater, storage, epochs: int, n_minibatches: int, perm: torch.Tensor = None):
    """The update phase over one collected rollout: `epochs` passes over `n_minibatches` blocks of the
    T * N samples (row t * N + e of the flattened time-major arrays).
    perm None: contiguous blocks -- each block's observations are converted into both nets' bf16 input
    rows by im_f32_to_bf16_padded, everything else is read in place from the storage.
    perm: int32 CUDA tensor [epochs, T * N], a permutation of the sample indices per epoch (shuffled
    minibatches): every per-sample array of a block is gathered by im_gather_rows_f32.
    Enqueues only; capturable in a CUDA graph together with the rollout."""
    T, N, A = storage.T, storage.N, storage.A
    total = T * N
    M = total // n_minibatches
    if total % n_minibatches or M % 64 or M > upd.Mb:
        raise ValueError("T * N must split into minibatches of a multiple of 64 rows that fit the trainers")
    if not storage.keep_obs:
        raise ValueError("the update reads the stored observations")
    flat = lambda x, *tail: x.view(total, *tail) if tail else x.view(total)
    obs = storage.obs[:T].view(total, storage.ld_obs)
    action, mean, logp = flat(storage.action, A), flat(storage.mean, A), flat(storage.logp)
    adv, ret, val = flat(storage.advantage), flat(storage.returns), storage.value[:T].reshape(total)
    D = upd.actor.dims[0]
    st = upd.stream
    if perm is not None:
        if perm.dtype != torch.int32 or tuple(perm.shape) != (epochs, total):
            raise ValueError("perm must be an int32 tensor [epochs, T * N]")
        if not hasattr(upd, "_gather") or upd._gather["action"].shape[0] < M:
            f = lambda *sh: torch.empty(*sh, dtype=torch.float32, device="cuda")
            upd._gather = dict(action=f(M, A), mean_old=f(M, A), logp_old=f(M), advantage=f(M), value_old=f(M), returns=f(M))
    for ep in range(epochs):
        for k in range(n_minibatches):
            sl = slice(k * M, (k + 1) * M)
            if perm is None:
                for tr in (upd.actor, upd.critic):
                    B.f32_to_bf16_padded(obs[sl, :D], tr.input_rows(M), st)
                batch = dict(action=action[sl], mean_old=mean[sl], logp_old=logp[sl], advantage=adv[sl], value_old=val[sl],
                             returns=ret[sl])
            else:
                idx = perm[ep, sl]
                for tr in (upd.actor, upd.critic):
                    B.gather_rows(obs[:, :D], idx, tr.input_rows(M), upd.actor.status, st)
                g = upd._gather
                for name, src in (("action", action), ("mean_old", mean), ("logp_old", logp), ("advantage", adv),
                                  ("value_old", val), ("returns", ret)):
                    B.gather_rows(src, idx, g[name][:M], upd.actor.status, st)
                batch = {name: g[name][:M] for name in g}
            upd.update(M, dict(batch, log_std_old=upd.log_std_old))


def _main():
    """python -m paper_2609_09821_b200.trainer [--rows M] [--passes P] [--dims 577 1024 1024 512 69]:
    forward + backward of one MLP on M random rows, P times; prints the time of the last pass."""
    import argparse
    from . import workloads as W
    ap = argparse.ArgumentParser()
    ap.add_argument("--rows", type=int, default=65536)
    ap.add_argument("--passes", type=int, default=2)
    ap.add_argument("--dims", type=int, nargs="+", default=[577, 1024, 1024, 512, 69])
    a = ap.parse_args()
    dims, M = tuple(a.dims), a.rows
    w = W.make_policy_weights(dims, "bf16", 1)
    tr = MlpTrainer(dims, w["W"], w["b"], M)
    gen = torch.Generator(device="cuda").manual_seed(0)
    rows = tr.input_rows(M)
    rows.zero_()
    rows[:, :dims[0]] = torch.randn((M, dims[0]), device="cuda", generator=gen).to(torch.bfloat16)
    d_out = torch.randn((M, dims[-1]), device="cuda", generator=gen) / M
    for _ in range(a.passes):
        e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        e[0].record(tr.stream); tr.forward(M)
        e[1].record(tr.stream); tr.backward(d_out, M)
        e[2].record(tr.stream); torch.cuda.synchronize()
    print("rows %d dims %s: forward %.3f ms, backward %.3f ms, device status %d"
          % (M, "-".join(map(str, dims)), e[0].elapsed_time(e[1]), e[1].elapsed_time(e[2]), tr.device_status()))


if __name__ == "__main__":
    _main()
