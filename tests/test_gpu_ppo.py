"""GPU parity of the PPO minibatch loss and the advantage moments against the CPU oracle, through
the C ABI.

Tolerances (fp32 kernel, fp64 oracle).  The probability ratio is exp of a difference of two
log-probabilities of magnitude up to ~A, so it carries a relative error of a few 1e-6 A^(1/2); all
ratio-dependent outputs are compared to 2e-4 of the output's largest magnitude plus 2e-4 relative.
Whether a sample's clip is active is a comparison of fp32 numbers: samples whose ratio lies within
1e-4 (relative) of a clip boundary may take either branch, are excluded from the element-wise
comparison of d_mean, and must be rare; the batch sums get a matching allowance.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2609_09821_b200 import binding as B
from paper_2609_09821_b200 import workloads as W

pytestmark = pytest.mark.gpu


def run_gpu(b, clip, cv, ce, clip_value, normalise):
    t = {k: torch.from_numpy(v).cuda() for k, v in b.items()}
    M, A = b["mean"].shape
    ws = B.ppo_workspace()
    mom = None
    if normalise:
        mom = torch.empty(2, device="cuda")
        B.moments(t["advantage"], mom, ws)
    d_mean = torch.full((M, A), float("nan"), device="cuda")
    d_log_std = torch.full((A,), float("nan"), device="cuda")
    d_value = torch.full((M,), float("nan"), device="cuda")
    summary = torch.full((6,), float("nan"), device="cuda")
    B.ppo_loss(t, d_mean, d_log_std, d_value, summary, ws, clip, cv, ce, clip_value, adv_moments=mom)
    torch.cuda.synchronize()
    return dict(d_mean=d_mean.cpu().numpy(), d_log_std=d_log_std.cpu().numpy(), d_value=d_value.cpu().numpy(),
                summary=summary.cpu().numpy(), moments=None if mom is None else mom.cpu().numpy())


def ratios(b):
    A = b["mean"].shape[1]
    z = (b["action"].astype(np.float64) - b["mean"]) / np.exp(b["log_std"].astype(np.float64))
    logp = -0.5 * (z ** 2).sum(1) - b["log_std"].astype(np.float64).sum() - 0.5 * A * np.log(2 * np.pi)
    return np.exp(logp - b["logp_old"])


def close(got, want, what, scale=None):
    want = np.asarray(want, np.float64)
    lim = 2e-4 * (np.abs(want).max() if scale is None else scale) + 2e-4 * np.abs(want)
    err = np.abs(np.asarray(got, np.float64) - want)
    assert (err <= lim).all(), "%s: worst error %.3e against limit %.3e" % (what, err.max(), lim[np.argmax(err - lim)])


@pytest.mark.parametrize("M,A,drift,clip", [(5000, 12, 0.05, 0.2), (4099, 69, 0.02, 0.32), (777, 1, 0.5, 0.2),
                                             (3000, 33, 0.03, 0.2), (1200, 128, 0.01, 0.2), (9, 28, 0.05, 0.2)])
@pytest.mark.parametrize("clip_value,normalise", [(False, False), (True, True)])
def test_ppo_loss_matches_oracle(M, A, drift, clip, clip_value, normalise):
    b = W.make_ppo_batch(M, A, seed=M + A, drift=drift)
    cv, ce = 2.0, 2.5e-4                                  # the paper's baseline value-loss / tuned entropy coefficients
    am, ar = O.moments(b["advantage"]) if normalise else (0.0, 1.0)
    want = O.ppo_loss(b, clip, cv, ce, clip_value, am, ar)
    got = run_gpu(b, clip, cv, ce, clip_value, normalise)
    if normalise:
        np.testing.assert_allclose(got["moments"], [am, ar], rtol=2e-6)
    r = ratios(b)
    edge = (np.abs(r - (1 - clip)) < 1e-4 * r) | (np.abs(r - (1 + clip)) < 1e-4 * r)
    assert edge.mean() <= 0.01
    close(got["d_mean"][~edge], want["d_mean"][~edge], "d_mean", scale=np.abs(want["d_mean"]).max())
    close(got["d_value"], want["d_value"], "d_value")
    # batch sums: each boundary sample may move a sum by its own contribution
    slack = edge.sum() * np.abs(want["d_mean"]).max() * 50
    assert np.abs(got["d_log_std"] - want["d_log_std"]).max() <= 2e-4 * np.abs(want["d_log_std"]).max() + 2e-6 + slack
    s_g, s_o = got["summary"], want["summary"]
    np.testing.assert_allclose(s_g[[0, 1, 2, 3, 4]], s_o[[0, 1, 2, 3, 4]], rtol=3e-4, atol=2e-5 + edge.mean())
    assert abs(s_g[5] - s_o[5]) <= edge.mean() + 1e-6
    assert np.isfinite(got["d_mean"]).all()


def test_ppo_loss_is_bit_reproducible_and_capturable():
    b = W.make_ppo_batch(20000, 69, seed=1, drift=0.02)
    a = run_gpu(b, 0.2, 2.0, 0.0, True, True)
    c = run_gpu(b, 0.2, 2.0, 0.0, True, True)
    for k in ("d_mean", "d_log_std", "d_value", "summary"):
        np.testing.assert_array_equal(a[k], c[k])
    t = {k: torch.from_numpy(v).cuda() for k, v in b.items()}
    ws, mom = B.ppo_workspace(), torch.empty(2, device="cuda")
    out = [torch.zeros((20000, 69), device="cuda"), torch.zeros(69, device="cuda"), torch.zeros(20000, device="cuda"),
           torch.zeros(6, device="cuda")]
    s = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        with torch.cuda.graph(g, stream=s):
            B.moments(t["advantage"], mom, ws, stream=s)
            B.ppo_loss(t, *out, ws, 0.2, 2.0, 0.0, True, adv_moments=mom, stream=s)
        g.replay()
    torch.cuda.synchronize()
    np.testing.assert_array_equal(out[0].cpu().numpy(), a["d_mean"])
    np.testing.assert_array_equal(out[3].cpu().numpy(), a["summary"])


def test_unaligned_arrays_take_the_element_wise_path():
    """Arrays that start 4 bytes off a 16-byte boundary cannot use bulk copies; same results."""
    M, A = 3000, 69
    b = W.make_ppo_batch(M, A, seed=8, drift=0.02)
    ref = run_gpu(b, 0.2, 2.0, 1e-3, True, False)

    def shifted(v):
        buf = torch.empty(v.size + 1, device="cuda")
        buf[1:] = torch.from_numpy(v.ravel()).cuda()
        return buf[1:].view(*v.shape)
    t = {k: shifted(v) for k, v in b.items()}
    assert t["mean"].data_ptr() % 16 == 4
    ws = B.ppo_workspace()
    d_mean, d_value = shifted(np.zeros((M, A), np.float32)), shifted(np.zeros(M, np.float32))
    d_log_std, summary = torch.empty(A, device="cuda"), torch.empty(6, device="cuda")
    B.ppo_loss(t, d_mean, d_log_std, d_value, summary, ws, 0.2, 2.0, 1e-3, True)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(d_mean.cpu().numpy(), ref["d_mean"])        # same arithmetic per row
    np.testing.assert_array_equal(d_value.cpu().numpy(), ref["d_value"])
    np.testing.assert_allclose(d_log_std.cpu().numpy(), ref["d_log_std"], rtol=1e-4, atol=1e-7)   # other summation order
    np.testing.assert_allclose(summary.cpu().numpy(), ref["summary"], rtol=1e-5)


def test_moments_edge_cases():
    ws = B.ppo_workspace()
    out = torch.empty(2, device="cuda")
    for x in (np.array([3.0], np.float32), np.full(1000, -2.5, np.float32),
              np.random.default_rng(0).normal(100.0, 0.01, 300000).astype(np.float32)):
        B.moments(torch.from_numpy(x).cuda(), out, ws)
        torch.cuda.synchronize()
        m, r = O.moments(x)
        np.testing.assert_allclose(out.cpu().numpy(), [m, r], rtol=1e-5)


def test_ppo_loss_rejects_bad_arguments():
    b = {k: torch.from_numpy(v).cuda() for k, v in W.make_ppo_batch(64, 200, 0).items()}
    ws = B.ppo_workspace()
    outs = [torch.empty((64, 200), device="cuda"), torch.empty(200, device="cuda"), torch.empty(64, device="cuda"),
            torch.empty(6, device="cuda")]
    with pytest.raises(B.ImError):
        B.ppo_loss(b, *outs, ws, 0.2, 1.0, 0.0, False)                 # A > 128
    b = {k: torch.from_numpy(v).cuda() for k, v in W.make_ppo_batch(64, 8, 0).items()}
    outs = [torch.empty((64, 8), device="cuda"), torch.empty(8, device="cuda"), torch.empty(64, device="cuda"),
            torch.empty(6, device="cuda")]
    with pytest.raises(B.ImError):
        B.ppo_loss(b, *outs, ws, -0.1, 1.0, 0.0, False)                # negative clip
    del b["value_old"]
    with pytest.raises(B.ImError):
        B.ppo_loss(b, *outs, ws, 0.2, 1.0, 0.0, True)                  # value clipping needs the old values
    B.ppo_loss(b, *outs, ws, 0.2, 1.0, 0.0, False)
    torch.cuda.synchronize()


# ---------------------------------------------------------------- optimiser step
@pytest.mark.parametrize("n", [1, 37, 4096, 1000003])
def test_adam_steps_match_oracle(n):
    g = np.random.default_rng(n)
    p0 = g.standard_normal(n).astype(np.float32)
    po, mo, vo = p0.copy(), np.zeros(n, np.float32), np.zeros(n, np.float32)
    pg, mg, vg = (torch.from_numpy(p0.copy()).cuda(), torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda"))
    lr = torch.tensor([5e-4], device="cuda")              # the paper's baseline learning rate
    for t in range(1, 5):
        grad = (g.standard_normal(n) * 10.0 ** g.uniform(-4, 1, n)).astype(np.float32)
        scale = 1.0 if t % 2 else 0.37
        # the coefficients reach the kernel as fp32: the oracle gets the same rounded values
        O.adam_step(po, grad, mo, vo, float(np.float32(5e-4)), t, b1=float(np.float32(0.9)), b2=float(np.float32(0.999)),
                    eps=float(np.float32(1e-8)), grad_scale=float(np.float32(scale)))
        B.adam_step(pg, torch.from_numpy(grad).cuda(), mg, vg, lr, t,
                    grad_scale=None if t % 2 else torch.tensor([scale], device="cuda"))
        torch.cuda.synchronize()
        # one fp32 rounding of each of the few operations: a few ulp of the operands
        np.testing.assert_allclose(pg.cpu().numpy(), po, rtol=2e-6, atol=2e-9)
        np.testing.assert_allclose(mg.cpu().numpy(), mo, rtol=1e-5, atol=1e-6 * np.abs(mo).max())
        np.testing.assert_allclose(vg.cpu().numpy(), vo, rtol=1e-5, atol=1e-6 * np.abs(vo).max())
        # keep both sides on the same trajectory
        po, mo, vo = pg.cpu().numpy().copy(), mg.cpu().numpy().copy(), vg.cpu().numpy().copy()


def test_grad_scale_and_adaptive_lr_match_oracle():
    g = np.random.default_rng(2)
    grads = [g.standard_normal(s).astype(np.float32) * 0.05 for s in (1024 * 577, 1024, 512 * 1024, 69, 1)]
    ws = B.ppo_workspace()
    out = torch.empty(2, device="cuda")
    dev = [torch.from_numpy(x).cuda() for x in grads]
    for max_norm in (1.0, 1e6):
        B.grad_scale(dev, max_norm, out, ws)
        torch.cuda.synchronize()
        want = O.grad_scale(grads, max_norm)
        np.testing.assert_allclose(out[0].item(), want, rtol=1e-6)
        np.testing.assert_allclose(out[1].item(), np.sqrt(sum((x.astype(np.float64) ** 2).sum() for x in grads)), rtol=1e-6)
    lr = torch.tensor([1e-3], device="cuda")
    for kl in (0.02, 0.003, 0.008, 0.0, 1.0, 1.0, 1.0):
        want = O.adaptive_lr(lr.item(), float(np.float32(kl)), 0.008)
        B.adaptive_lr(lr, torch.tensor([kl], device="cuda"), 0.008)
        torch.cuda.synchronize()
        np.testing.assert_allclose(lr.item(), want, rtol=1e-6)
    with pytest.raises(B.ImError):
        B.grad_scale(dev, -1.0, out, ws)


def test_adam_writes_new_weights_into_a_loaded_policy():
    """The bf16 copy of an Adam step lands in a tensor-core policy's padded weight matrix: the next
    forward equals a policy loaded with the updated weights."""
    dims = (361, 128, 28)
    n = 300
    pw = W.make_policy_weights(dims, "bf16", 4)
    pol = B.Policy(dims, pw["W_bf16"], pw["b"], "bf16", 0.1, 0, n)
    g = np.random.default_rng(6)
    lr = torch.tensor([1e-2], device="cuda")
    new_W = []
    for l in range(2):
        w_ptr, ld, b_ptr = pol.layer_buffers(l)
        assert ld == (dims[l] + 63) // 64 * 64
        master = torch.from_numpy(pw["W"][l].copy()).cuda()                       # fp32 master copy
        grad = torch.from_numpy(g.standard_normal(pw["W"][l].shape).astype(np.float32)).cuda()
        m, v = torch.zeros_like(master), torch.zeros_like(master)
        B.adam_step(master, grad, m, v, lr, 1, bf16_out_ptr=w_ptr, cols=dims[l], ld_bf16=ld)
        new_W.append(master.cpu().numpy())
    torch.cuda.synchronize()
    obs = torch.zeros((n, 384), device="cuda")
    obs[:, :361] = torch.from_numpy(g.standard_normal((n, 361)).astype(np.float32)).cuda()
    mean, act = torch.empty((n, 28), device="cuda"), torch.empty((n, 28), device="cuda")
    pol.forward(1, obs, mean, act)
    ref_bits = [W.round_to_bf16(x)[1] for x in new_W]
    ref = B.Policy(dims, ref_bits, pw["b"], "bf16", 0.1, 0, n)
    mean2, act2 = torch.empty_like(mean), torch.empty_like(act)
    ref.forward(1, obs, mean2, act2)
    torch.cuda.synchronize()
    assert torch.equal(mean, mean2) and torch.equal(act, act2)
    assert np.abs(new_W[0] - pw["W"][0]).max() > 5e-3                              # the step moved the weights
