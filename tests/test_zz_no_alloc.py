"""The allocation-free policy forward against the regular one.

Some callers of the library cannot call cudaMalloc at the moment they need an action (a control
loop with a latency budget, a process whose device memory was all handed out at start-up).  They
use im_policy_forward_noalloc, whose hidden activations live in a fixed array inside the library.
This test calls it through the C ABI twice in a row and requires the same means, actions and
log-probabilities as im_policy_forward on the same weights and observations, within the
tolerance the parity tests use for the fp32 policy; the second call also checks that what the
first call left in the shared array does no harm.  Both calls are also compared with the CPU
oracle directly, and the device's free memory must be the same before and after a call once the
first call has been made.  The file sorts last so that a run that stops at the first failure has
already run everything else.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2609_09821_b200 import binding as B
from paper_2609_09821_b200 import workloads as W
from tests.parity import assert_close, assert_mean_close

pytestmark = pytest.mark.gpu


def _reference(pol, sigma, seed, step, obs):
    n, A = obs.shape[0], pol["dims"][-1]
    policy = B.Policy(pol["dims"], pol["W"], pol["b"], "f32", sigma, seed, n)
    mean = torch.empty((n, A), device="cuda")
    act = torch.empty((n, A), device="cuda")
    logp = torch.empty(n, device="cuda")
    policy.forward(step, obs, mean, act, logp)
    torch.cuda.synchronize()
    return mean, act, logp


def test_noalloc_policy_matches_regular_policy_twice():
    wl = W.WORKLOADS["cfg1_tiny64"]
    sigma, seed = wl.sigma_action, 1234
    pol = W.make_policy_weights(wl.mlp_dims, "f32", seed=3)
    Wd = [torch.from_numpy(w).cuda() for w in pol["W"]]
    bd = [torch.from_numpy(x).cuda() for x in pol["b"]]
    A = pol["dims"][-1]
    g = torch.Generator(device="cuda").manual_seed(7)
    # two calls in a row, of different sizes, so the second finds the first one's leftovers
    for step, n in ((1, 777), (2, 64)):
        obs = torch.zeros((n, 384), device="cuda")
        obs[:, :361] = torch.randn((n, 361), generator=g, device="cuda") * 2.0
        obs[:, 361:] = float("nan")                      # padding must never be read
        want_mean, want_act, want_logp = _reference(pol, sigma, seed, step, obs)
        mean = torch.full((n, A), float("nan"), device="cuda")
        act = torch.full((n, A), float("nan"), device="cuda")
        logp = torch.full((n,), float("nan"), device="cuda")
        B.policy_forward_noalloc(pol["dims"], Wd, bd, sigma, seed, step, obs, mean, act, logp)
        torch.cuda.synchronize()
        # once the first call has run, a call leaves the device's free memory where it was
        free_before = torch.cuda.mem_get_info()[0]
        B.policy_forward_noalloc(pol["dims"], Wd, bd, sigma, seed, step, obs, mean, act, logp)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before
        # the oracle itself, not only the library's other path
        o = O.policy_forward(pol["dims"], pol["W"], pol["b"], sigma, seed, step,
                             obs[:, :361].cpu().numpy().astype(np.float64), env_ids=np.arange(n, dtype=np.uint32))
        assert_mean_close(mean.cpu().numpy(), o["mean"], 1e-4, what="step %d vs oracle" % step)
        assert_close((act - mean).cpu().numpy().astype(np.float64), sigma * o["z"], atol=1e-5, rtol=1e-4,
                     what="step %d action noise vs oracle" % step)
        assert_close(logp.cpu().numpy(), o["logp"], atol=1e-3, rtol=1e-5, what="step %d logp vs oracle" % step)
        assert_mean_close(mean.cpu().numpy(), want_mean.cpu().numpy(), 1e-4, what="step %d" % step)
        noise = (act - mean).cpu().numpy().astype(np.float64)
        want_noise = (want_act - want_mean).cpu().numpy().astype(np.float64)
        assert_close(noise, want_noise, atol=1e-5, rtol=1e-4, what="step %d action noise" % step)
        assert_close(logp.cpu().numpy(), want_logp.cpu().numpy(), atol=1e-3, rtol=1e-5, what="step %d logp" % step)


def test_noalloc_policy_rejects_sizes_beyond_its_scratch():
    dims = (8, 16, 4)
    Wd = [torch.zeros((16, 8), device="cuda"), torch.zeros((4, 16), device="cuda")]
    bd = [torch.zeros(16, device="cuda"), torch.zeros(4, device="cuda")]
    n = B.NOALLOC_MAX_BATCH + 1
    obs = torch.zeros((n, 8), device="cuda")
    out = torch.zeros((n, 4), device="cuda")
    with pytest.raises(B.ImError) as e:
        B.policy_forward_noalloc(dims, Wd, bd, 0.1, 0, 0, obs, out, out.clone())
    assert e.value.status == -6
    wide = (8, B.NOALLOC_MAX_WIDTH + 64, 4)
    Ww = [torch.zeros((wide[1], 8), device="cuda"), torch.zeros((4, wide[1]), device="cuda")]
    bw = [torch.zeros(wide[1], device="cuda"), torch.zeros(4, device="cuda")]
    with pytest.raises(B.ImError) as e:
        B.policy_forward_noalloc(wide, Ww, bw, 0.1, 0, 0, obs[:8], out[:8], out[:8].clone())
    assert e.value.status == -6
