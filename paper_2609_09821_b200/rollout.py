"""Rollout storage and collection on top of the C-ABI calls (argument marshalling only).

The training loop of the paper's Figure 2 writes obs, action, reward, terminated and truncated into
a storage object every step and hands it to the PPO update.  Here the storage is a set of
time-major device arrays and "writing" costs nothing: each per-step call is given pointers into
row t of the arrays, so the env kernel and the policy head store their results in place.
After the last step the critic evaluates the final observation and one im_gae launch fills the
advantages and returns.
"""
from __future__ import annotations

from typing import Callable, Optional

import torch

from . import binding as B


class RolloutStorage:
    """Device arrays of one rollout: T control steps of N envs.

    obs      [T + 1, N, ld_obs] float32   (row t is what the policy saw at step t; optional)
    action   [T, N, A]   mean [T, N, A]   logp [T, N]
    value    [T + 1, N]  reward [T, N]    flags [T, N] uint8 (bit 0 terminated, bit 1 truncated)
    advantage, returns [T, N]
    """

    def __init__(self, T: int, N: int, A: int, ld_obs: int, keep_obs: bool = True, device="cuda"):
        self.T, self.N, self.A, self.ld_obs = T, N, A, ld_obs
        f32 = dict(dtype=torch.float32, device=device)
        # without obs history two rows are enough: the env writes row (t + 1) % 2 while row t % 2 is read
        self.obs = torch.zeros((T + 1 if keep_obs else 2, N, ld_obs), **f32)
        self.keep_obs = keep_obs
        self.action = torch.empty((T, N, A), **f32)
        self.mean = torch.empty((T, N, A), **f32)
        self.logp = torch.empty((T, N), **f32)
        self.value = torch.empty((T + 1, N), **f32)
        self.reward = torch.empty((T, N), **f32)
        self.flags = torch.empty((T, N), dtype=torch.uint8, device=device)
        self.advantage = torch.empty((T, N), **f32)
        self.returns = torch.empty((T, N), **f32)

    def obs_row(self, t: int) -> torch.Tensor:
        return self.obs[t if self.keep_obs else t % 2]


def collect(env: B.Env, actor: B.Policy, critic: Optional[B.Policy], storage: RolloutStorage,
            sim_of_step: Callable[[int], torch.Tensor], step0: int, gamma: float, lam: float,
            bootstrap_truncated: bool = True, staged: bool = False):
    """Runs T control steps from the env's current state and fills `storage`.

    storage.obs_row(0) must hold the current observation (from Env.reset_all or the previous
    rollout's last row).  sim_of_step(s) returns the simulator's body states after the physics of
    global step s (a CUDA tensor [13 J, stride]).  With staged=True the env must be attached to
    the actor; actor and critic then read the bf16 rows the env kernel leaves in the actor's input
    buffer.  Everything is enqueued on the env's stream; nothing here waits for the device, so the
    whole call can be captured in a CUDA graph.
    """
    st, T, N = storage, storage.T, storage.N
    for t in range(T):
        s = step0 + t
        obs = st.obs_row(t)
        if staged:
            actor.forward_staged(s, N, st.mean[t], st.action[t], st.logp[t])
            if critic is not None:
                critic.value_forward_staged(N, st.value[t].unsqueeze(1), src=actor)
        else:
            actor.forward(s, obs, st.mean[t], st.action[t], st.logp[t])
            if critic is not None:
                critic.value_forward(obs, st.value[t].unsqueeze(1))
        if getattr(env, "_prev_action", None) is not None:
            # extended observation: the next row's previous-action entries are this step's actions (host state
            # only; the pointer travels with the launch, so a captured graph keeps one per step)
            env.set_obs_extension(env.n_future, st.action[t])
        env.step(s, sim_of_step(s), st.obs_row(t + 1), st.reward[t], st.flags[t])
    if critic is not None:
        last = st.obs_row(T)
        if staged:
            critic.value_forward_staged(N, st.value[T].unsqueeze(1), src=actor)
        else:
            critic.value_forward(last, st.value[T].unsqueeze(1))
        B.gae(st.reward, st.value, st.flags, st.advantage, st.returns, gamma, lam, bootstrap_truncated,
              stream=env.stream)
