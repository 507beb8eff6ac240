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


# ---------------------------------------------------------------- optimiser step
def test_adam_matches_torch_optim_over_several_steps():
    g = np.random.default_rng(0)
    n = 5000
    p0 = g.standard_normal(n).astype(np.float32)
    grads = [(g.standard_normal(n) * 10.0 ** g.uniform(-4, 1, n)).astype(np.float32) for _ in range(6)]
    p, m, v = p0.copy(), np.zeros(n, np.float32), np.zeros(n, np.float32)
    tp = torch.nn.Parameter(torch.tensor(p0, dtype=torch.float64))
    opt = torch.optim.Adam([tp], lr=5e-4, betas=(0.9, 0.999), eps=1e-8)
    for t, gr in enumerate(grads, 1):
        O.adam_step(p, gr, m, v, 5e-4, t)
        tp.grad = torch.tensor(gr, dtype=torch.float64)
        opt.step()
        # the oracle stores its state in fp32 between steps: agreement to fp32 rounding
        np.testing.assert_allclose(p, tp.detach().numpy(), rtol=1e-6, atol=1e-7)
    st = opt.state[tp]
    # state kept in fp32 between steps: errors of one fp32 rounding of the largest summand
    np.testing.assert_allclose(m, st["exp_avg"].numpy(), rtol=1e-5, atol=1e-6 * np.abs(m).max())
    np.testing.assert_allclose(v, st["exp_avg_sq"].numpy(), rtol=1e-5, atol=1e-6 * np.abs(v).max())


def test_adam_first_step_moves_by_lr_against_the_gradient_sign():
    grad = np.array([3.0, -0.5, 1e-3, -40.0], np.float32)
    p, m, v = np.zeros(4, np.float32), np.zeros(4, np.float32), np.zeros(4, np.float32)
    O.adam_step(p, grad, m, v, 1e-2, 1)
    np.testing.assert_allclose(p, -1e-2 * np.sign(grad), rtol=1e-4)       # m_hat / sqrt(v_hat) = sign(g) at t = 1
    np.testing.assert_allclose(m, 0.1 * grad, rtol=1e-6)
    np.testing.assert_allclose(v, 0.001 * grad.astype(np.float64) ** 2, rtol=1e-6)
    q, m2, v2 = np.zeros(4, np.float32), np.zeros(4, np.float32), np.zeros(4, np.float32)
    O.adam_step(q, grad, m2, v2, 1e-2, 1, grad_scale=0.25)               # scaling g leaves the first step unchanged
    np.testing.assert_allclose(q, p, rtol=1e-4)
    np.testing.assert_allclose(m2, 0.25 * m, rtol=1e-6)


def test_grad_scale_matches_torch_clip_grad_norm():
    g = np.random.default_rng(1)
    grads = [g.standard_normal(s).astype(np.float32) * 0.3 for s in ((40, 7), (7,), (300,))]
    for max_norm in (1.0, 100.0):
        params = [torch.nn.Parameter(torch.zeros(x.shape, dtype=torch.float64)) for x in grads]
        for prm, x in zip(params, grads):
            prm.grad = torch.tensor(x, dtype=torch.float64)
        total = torch.nn.utils.clip_grad_norm_(params, max_norm)
        s = O.grad_scale(grads, max_norm)
        np.testing.assert_allclose(s, min(1.0, max_norm / (total.item() + 1e-6)), rtol=1e-12)
        np.testing.assert_allclose(params[0].grad.numpy(), grads[0].astype(np.float64) * s, rtol=1e-9)
    assert O.grad_scale(grads, 100.0) == 1.0


def test_adaptive_learning_rate_rule():
    kl_t = 0.008                                          # the paper's baseline KL threshold
    assert O.adaptive_lr(1e-3, 0.02, kl_t) == pytest.approx(1e-3 / 1.5)
    assert O.adaptive_lr(1e-3, 0.003, kl_t) == pytest.approx(1.5e-3)
    assert O.adaptive_lr(1e-3, 0.008, kl_t) == 1e-3
    assert O.adaptive_lr(1e-3, 0.0, kl_t) == 1e-3         # no information: unchanged
    assert O.adaptive_lr(1.2e-5, 1.0, kl_t) == 1e-5       # clamped below
    assert O.adaptive_lr(9e-3, 1e-6, kl_t) == 1e-2        # clamped above


# ---------------------------------------------------------------- backward pass of the MLP
def test_mlp_backward_matches_torch_autograd():
    g = np.random.default_rng(3)
    dims = (23, 40, 32, 7)
    Ws = [g.standard_normal((o, i)).astype(np.float32) / math.sqrt(i) for i, o in zip(dims[:-1], dims[1:])]
    bs = [g.standard_normal(o).astype(np.float32) * 0.1 for o in dims[1:]]
    obs = g.standard_normal((50, 23))
    g_out = g.standard_normal((50, 7))
    dW, db = O.mlp_backward(dims, Ws, bs, obs, g_out)
    tW = [torch.tensor(w, dtype=torch.float64, requires_grad=True) for w in Ws]
    tb = [torch.tensor(x, dtype=torch.float64, requires_grad=True) for x in bs]
    h = torch.tensor(obs)
    for l in range(3):
        h = torch.nn.functional.linear(h, tW[l], tb[l])
        if l < 2:
            h = torch.relu(h)
    (h * torch.tensor(g_out)).sum().backward()
    for l in range(3):
        np.testing.assert_allclose(dW[l], tW[l].grad.numpy(), rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(db[l], tb[l].grad.numpy(), rtol=1e-10, atol=1e-12)
    # bf16 weights and operands move the gradients (masks near zero flip), but not far; dW comes out as bf16 values
    dWb, dbb = O.mlp_backward(dims, [W.round_to_bf16(w)[0] for w in Ws], bs, obs, g_out, bf16_operands=True)
    for l in range(3):
        scale = np.abs(dW[l]).max()
        assert 1e-6 * scale < np.abs(dWb[l] - dW[l]).max() < 0.2 * scale
        np.testing.assert_array_equal(dWb[l], W.round_to_bf16(dWb[l].astype(np.float32))[0])


def test_mlp_backward_single_linear_layer_closed_form():
    """One layer, no activation: dW = g^T x, db = column sums of g."""
    g = np.random.default_rng(4)
    Wm = g.standard_normal((5, 9)).astype(np.float32)
    x, go = g.standard_normal((13, 9)), g.standard_normal((13, 5))
    dW, db = O.mlp_backward((9, 5), [Wm], [np.zeros(5, np.float32)], x, go)
    np.testing.assert_allclose(dW[0], go.T @ x, rtol=1e-12)
    np.testing.assert_allclose(db[0], go.sum(0), rtol=1e-12)
