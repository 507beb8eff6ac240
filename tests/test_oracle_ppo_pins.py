"""Pins for the oracle's PPO minibatch loss: the same objective written with torch's distribution
and autograd routines in fp64 (an independent library computation of every gradient), plus special
cases with closed forms."""
import math

import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2609_09821_b200 import workloads as W


def torch_ppo(batch, clip, cv, ce, clip_value, adv_mean, adv_rstd):
    t = {k: torch.tensor(np.asarray(v, np.float32), dtype=torch.float64) for k, v in batch.items()}
    mean = t["mean"].clone().requires_grad_(True)
    log_std = t["log_std"].clone().requires_grad_(True)
    value = t["value"].clone().requires_grad_(True)
    dist = torch.distributions.Normal(mean, log_std.exp().expand_as(mean))
    logp = dist.log_prob(t["action"]).sum(-1)
    ratio = (logp - t["logp_old"]).exp()
    ah = (t["advantage"] - adv_mean) * adv_rstd
    surr = -torch.min(ratio * ah, ratio.clamp(1 - clip, 1 + clip) * ah)
    if clip_value:
        vc = t["value_old"] + (value - t["value_old"]).clamp(-clip, clip)
        vl = torch.max((value - t["returns"]) ** 2, (vc - t["returns"]) ** 2)
    else:
        vl = (value - t["returns"]) ** 2
    ent = dist.entropy().sum(-1)
    loss = surr.mean() + cv * vl.mean() - ce * ent.mean()
    loss.backward()
    old = torch.distributions.Normal(t["mean_old"], t["log_std_old"].exp().expand_as(mean))
    kl = torch.distributions.kl_divergence(old, torch.distributions.Normal(mean.detach(), log_std.detach().exp().expand_as(mean)))
    return dict(d_mean=mean.grad.numpy(), d_log_std=log_std.grad.numpy(), d_value=value.grad.numpy(),
                summary=np.array([loss.item(), surr.mean().item(), vl.mean().item(), ent.mean().item(),
                                  kl.sum(-1).mean().item(), ((ratio - 1).abs() > clip).double().mean().item()]))


@pytest.mark.parametrize("clip_value", [False, True])
@pytest.mark.parametrize("A,drift,clip", [(12, 0.05, 0.2), (69, 0.02, 0.32), (1, 0.5, 0.2)])
def test_loss_and_gradients_match_torch_autograd(A, drift, clip, clip_value):
    M = 700
    b = W.make_ppo_batch(M, A, seed=A, drift=drift)
    am, ar = O.moments(b["advantage"])
    got = O.ppo_loss(b, clip, 2.0, 2.5e-4, clip_value, am, ar)
    want = torch_ppo(b, clip, 2.0, 2.5e-4, clip_value, am, ar)
    for k in ("d_mean", "d_log_std", "d_value", "summary"):
        # sums of M terms with cancellation: agreement to ~1e-9 of the largest entry
        np.testing.assert_allclose(got[k], want[k], rtol=1e-8, atol=1e-9 * np.abs(want[k]).max(), err_msg=k)
    assert 0.02 < got["summary"][5] < 0.9                  # clipped and unclipped samples both present


def test_moments_match_torch():
    x = W.make_ppo_batch(5000, 2, 1)["advantage"]
    m, r = O.moments(x)
    t = torch.tensor(x, dtype=torch.float64)
    np.testing.assert_allclose(m, t.mean().item(), rtol=1e-12)
    np.testing.assert_allclose(r, 1.0 / (t.std().item() + 1e-8), rtol=1e-12)
    assert O.moments(np.array([3.0], np.float32)) == (3.0, 1e8)


def test_unchanged_policy_closed_forms():
    """Current = behaviour policy: every ratio is 1, the surrogate is minus the mean advantage, the KL
    is 0, nothing is clipped, and dL/dmu = -Ahat (a - mu) / (sigma^2 M)."""
    M, A = 300, 7
    b = W.make_ppo_batch(M, A, 3, drift=0.0)
    b["mean"] = b["mean_old"].copy()
    b["log_std"] = b["log_std_old"].copy()
    # logp_old as the generator stored it (fp32) differs from the exact value by rounding only
    out = O.ppo_loss(b, 0.2, 0.0, 0.0, False)
    np.testing.assert_allclose(out["summary"][1], -b["advantage"].astype(np.float64).mean(), rtol=1e-4)
    assert abs(out["summary"][4]) < 1e-12 and out["summary"][5] == 0.0
    sg = np.exp(b["log_std"].astype(np.float64))
    want = -b["advantage"].astype(np.float64)[:, None] * (b["action"].astype(np.float64) - b["mean"]) / sg ** 2 / M
    np.testing.assert_allclose(out["d_mean"], want, rtol=2e-4, atol=1e-12)
    np.testing.assert_allclose(out["summary"][3], (b["log_std"].astype(np.float64) + 0.5 * math.log(2 * math.pi * math.e)).sum())


def test_clipped_samples_have_no_policy_gradient():
    M, A = 400, 5
    b = W.make_ppo_batch(M, A, 4, drift=0.3)
    out = O.ppo_loss(b, 0.2, 1.0, 0.0, False)
    sg = np.exp(b["log_std"].astype(np.float64))
    z = (b["action"].astype(np.float64) - b["mean"]) / sg
    logp = -0.5 * (z ** 2).sum(1) - b["log_std"].astype(np.float64).sum() - 0.5 * A * math.log(2 * math.pi)
    r = np.exp(logp - b["logp_old"])
    adv = b["advantage"].astype(np.float64)
    dead = ((r > 1.2) & (adv > 0)) | ((r < 0.8) & (adv < 0))           # the clip is active and binds
    assert dead.sum() > 20 and (~dead).sum() > 20
    assert np.all(out["d_mean"][dead] == 0.0)
    assert np.all(np.abs(out["d_mean"][~dead]).sum(axis=1) > 0.0)
    # value part: plain squared error
    np.testing.assert_allclose(out["d_value"], 2.0 * (b["value"].astype(np.float64) - b["returns"]) / M, rtol=1e-12)


def test_entropy_coefficient_only_moves_log_std():
    b = W.make_ppo_batch(200, 6, 5)
    a = O.ppo_loss(b, 0.2, 1.0, 0.0, True)
    c = O.ppo_loss(b, 0.2, 1.0, 0.01, True)
    np.testing.assert_array_equal(a["d_mean"], c["d_mean"])
    np.testing.assert_array_equal(a["d_value"], c["d_value"])
    ce = float(np.float32(0.01))                         # the coefficient travels as fp32
    np.testing.assert_allclose(c["d_log_std"] - a["d_log_std"], -ce, rtol=1e-9)
    np.testing.assert_allclose(c["summary"][0] - a["summary"][0], -ce * a["summary"][3], rtol=1e-9)
