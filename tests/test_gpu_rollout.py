"""GPU parity of the rollout-side calls (value head, advantage estimation) against the CPU oracle,
through the C ABI.

Tolerance of the advantage estimator (fp32 kernel vs fp64 oracle): one step of the recursion
A_t = delta_t + c_t A_{t+1} adds a rounding error of at most 3 u M (u = 2^-24; M bounds |reward| +
|value| + |A|) and damps the error carried in by c_t <= gamma lambda, so the error of any A_t is at
most 3 u M min(T, 1 / (1 - gamma lambda)); the chunked evaluation composes the same maps and obeys the
same bound.  The test allows four times that.
"""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2609_09821_b200 import binding as B
from paper_2609_09821_b200 import workloads as W
from tests.parity import Pair, Scene, assert_mean_close

pytestmark = pytest.mark.gpu

U = 2.0 ** -24


def gae_tolerance(T, gamma, lam, reward, value, adv):
    span = min(float(T), 1.0 / max(1.0 - gamma * lam, 1e-9))
    M = np.abs(reward).max() + np.abs(value).max() + np.abs(adv).max()
    return 4.0 * 3.0 * U * M * span


def run_gae(reward, value, flags, gamma, lam, bootstrap=True, ld=None):
    T, N = reward.shape
    ld = N if ld is None else ld
    dev = "cuda"

    def up(a, rows, dtype):
        buf = torch.full((rows, ld), 77, dtype=dtype, device=dev)
        buf[:, :N] = torch.from_numpy(a).to(dev)
        return buf
    r, v, f = up(reward, T, torch.float32), up(value, T + 1, torch.float32), up(flags, T, torch.uint8)
    adv = torch.full((T, ld), -12345.0, device=dev)
    ret = torch.full((T, ld), -12345.0, device=dev)
    B.gae(r[:, :N], v[:, :N], f[:, :N], adv[:, :N], ret[:, :N], gamma, lam, bootstrap)
    torch.cuda.synchronize()
    return adv.cpu().numpy(), ret.cpu().numpy()


@pytest.mark.parametrize("T,N,ld", [(32, 4096 + 17, None), (1, 5, None), (8, 33, 48), (7, 100, None), (13, 64, 64),
                                     (129, 70, 96), (200, 257, None), (300, 31, None),
                                     # aligned row strides and env counts that are multiples of four
                                     (32, 4096 + 16, None), (200, 256, 320), (1, 4, None), (9, 132, 136)])
@pytest.mark.parametrize("gamma,lam,bootstrap", [(0.99, 0.95, True), (0.98, 0.99, False)])
def test_gae_matches_oracle(T, N, ld, gamma, lam, bootstrap):
    """Horizons that are not a multiple of the 8-step chunk, several 128-step windows, ragged env
    tiles, padded rows; the paper's baseline and tuned (discount, lambda) pairs."""
    reward, value, flags = W.make_rollout_signals(T, N, seed=T * 1000 + N, p_term=0.03, p_trunc=0.03)
    adv_o, ret_o = O.gae(reward, value, flags, gamma, lam, bootstrap)
    adv_g, ret_g = run_gae(reward, value, flags, gamma, lam, bootstrap, ld)
    tol = gae_tolerance(T, gamma, lam, reward, value, adv_o)
    assert np.abs(adv_g[:, :N] - adv_o).max() <= tol
    assert np.abs(ret_g[:, :N] - ret_o).max() <= tol
    if ld is not None and ld > N:                        # padding columns are not written
        assert (adv_g[:, N:] == -12345.0).all() and (ret_g[:, N:] == -12345.0).all()


def test_gae_edge_cases():
    T, N = 24, 40
    reward, value, _ = W.make_rollout_signals(T, N, seed=3)
    for name, flags in (("no episode ends", np.zeros((T, N), np.uint8)),
                        ("every step terminates", np.ones((T, N), np.uint8)),
                        ("every step truncates", np.full((T, N), 2, np.uint8)),
                        ("both bits", np.full((T, N), 3, np.uint8))):
        for gamma, lam in ((0.99, 0.95), (1.0, 1.0), (0.0, 0.5), (0.9, 0.0)):
            adv_o, ret_o = O.gae(reward, value, flags, gamma, lam, True)
            adv_g, ret_g = run_gae(reward, value, flags, gamma, lam, True)
            tol = gae_tolerance(T, gamma, lam, reward, value, adv_o)
            assert np.abs(adv_g - adv_o).max() <= tol, (name, gamma, lam)
            assert np.abs(ret_g - ret_o).max() <= tol, (name, gamma, lam)


def test_gae_full_size_and_graph_capture():
    """The benchmark's rollout: 32 steps of 65536 envs, every element against the oracle; then the
    same launch replayed from a CUDA graph."""
    T, N = 32, 65536
    reward, value, flags = W.make_rollout_signals(T, N, seed=0)
    adv_o, ret_o = O.gae(reward, value, flags, 0.99, 0.95, True)
    r, v, f = (torch.from_numpy(a).cuda() for a in (reward, value, flags))
    adv, ret = torch.empty((T, N), device="cuda"), torch.empty((T, N), device="cuda")
    B.gae(r, v, f, adv, ret, 0.99, 0.95, True)
    torch.cuda.synchronize()
    tol = gae_tolerance(T, 0.99, 0.95, reward, value, adv_o)
    assert np.abs(adv.cpu().numpy() - adv_o).max() <= tol
    assert np.abs(ret.cpu().numpy() - ret_o).max() <= tol
    first = adv.clone()
    s = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        adv.zero_()
        with torch.cuda.graph(g, stream=s):
            B.gae(r, v, f, adv, ret, 0.99, 0.95, True, stream=s)
        g.replay()
    torch.cuda.synchronize()
    assert torch.equal(adv, first)


def test_gae_rejects_bad_arguments():
    r = torch.zeros((4, 8), device="cuda")
    v = torch.zeros((5, 8), device="cuda")
    f = torch.zeros((4, 8), dtype=torch.uint8, device="cuda")
    a, q = torch.empty_like(r), torch.empty_like(r)
    for gamma, lam in ((1.5, 0.9), (0.9, -0.1), (float("nan"), 0.5)):
        with pytest.raises(B.ImError):
            B.gae(r, v, f, a, q, gamma, lam)
    with pytest.raises(ValueError):
        B.gae(r, v[:4], f, a, q, 0.9, 0.9)


# ---------------------------------------------------------------- value head
def critic_weights(in_dim, dtype, seed=7):
    return W.make_policy_weights((in_dim, 512, 256, 1), dtype, seed)


@pytest.mark.parametrize("dtype,n", [("f32", 300), ("bf16", 300), ("bf16", 4096 + 5)])
def test_value_head_matches_oracle(dtype, n):
    cw = critic_weights(361, dtype)
    g = np.random.default_rng(11)
    obs = g.standard_normal((n, 361)).astype(np.float32)
    want = O.policy_forward(cw["dims"], cw["W"], cw["b"], 1.0, 0, 0, obs.astype(np.float64),
                            bf16_operands=dtype == "bf16")["mean"]
    critic = B.Policy(cw["dims"], cw["W_bf16"] if dtype == "bf16" else cw["W"], cw["b"], dtype, 1.0, 0, n)
    obs_g = torch.zeros((n, 384), device="cuda")
    obs_g[:, :361] = torch.from_numpy(obs).cuda()
    value = torch.full((n, 1), float("nan"), device="cuda")
    critic.value_forward(obs_g, value)
    torch.cuda.synchronize()
    assert_mean_close(value.cpu().numpy(), want, 2e-2 if dtype == "bf16" else 1e-4, "value head")
    # the same network through the sampling call gives the same means; without an action buffer no noise is drawn
    mean = torch.empty((n, 1), device="cuda")
    act = torch.empty((n, 1), device="cuda")
    critic.forward(5, obs_g, mean, act)
    mean2 = torch.empty((n, 1), device="cuda")
    critic.forward(5, obs_g, mean2, None)
    torch.cuda.synchronize()
    assert torch.equal(mean, value) and torch.equal(mean2, value)
    assert critic.device_status() == 0


def test_value_head_on_rows_staged_by_the_env():
    """The env writes bf16 observation rows into the actor's input buffer; the critic reads the same
    rows: equal, bit for bit, to the critic run on the fp32 observations, and close to the oracle."""
    sc = Scene(W.WORKLOADS["cfg3_16384_lib32"])
    n = 1000
    p = Pair(sc, n)
    cw = critic_weights(361, "bf16")
    critic = B.Policy(cw["dims"], cw["W_bf16"], cw["b"], "bf16", 1.0, 0, n)
    p.g_env.attach_policy(p.policy)
    p.reset_all()
    v_staged = torch.empty((n, 1), device="cuda")
    v_plain = torch.empty((n, 1), device="cuda")
    for s in (1, 2):
        critic.value_forward_staged(n, v_staged, src=p.policy)
        critic.value_forward(p.obs_g, v_plain)
        torch.cuda.synchronize()
        assert torch.equal(v_staged, v_plain)
        want = O.policy_forward(cw["dims"], cw["W"], cw["b"], 1.0, 0, 0, p.obs_o[:, :361].astype(np.float64),
                                bf16_operands=True)["mean"]
        assert_mean_close(v_staged.cpu().numpy(), want, 2e-2, "staged value head")
        sim = W.synth_sim_state_torch(sc.skel, sc.lib, torch.from_numpy(p.o_env.clip_id.astype(np.int64)),
                                      torch.from_numpy(p.o_env.t.astype(np.float64)) + sc.wl.dt, s, sc.wl)
        p.env_step(s, sim)
    p.g_env.attach_policy(None)
    # a critic of another input width cannot read the actor's rows
    other = critic_weights(577, "bf16")
    bad = B.Policy(other["dims"], other["W_bf16"], other["b"], "bf16", 1.0, 0, n)
    with pytest.raises(B.ImError):
        bad.value_forward_staged(n, v_staged, src=p.policy)


# ---------------------------------------------------------------- whole rollout into storage
@pytest.mark.parametrize("staged", [False, True], ids=["fp32-rows", "staged-bf16-rows"])
def test_collect_fills_storage_like_the_separate_calls(staged):
    """T steps collected straight into time-major storage: every stored signal against the oracle
    stage by stage, and the advantages against the oracle's estimator fed the stored signals."""
    from paper_2609_09821_b200 import rollout as R
    from tests.parity import assert_close
    wl = W.WORKLOADS["cfg3_16384_lib32"]
    sc = Scene(wl)
    n, T, gamma, lam = 512, 6, 0.99, 0.95
    ld = B.padded_ld(wl.obs_dim)
    pol = sc.pol
    cw = critic_weights(wl.obs_dim, "bf16")
    o_env = O.Env(sc.o_skel, sc.o_clips, O.make_env_config(wl.dt, 0, W.REWARD_MULT, 0.8), n)
    g_env = B.Env(sc.g_skel, sc.g_clips, B.make_env_config(n, wl.dt, 0, W.REWARD_MULT, 0.8, ld))
    actor = B.Policy(pol["dims"], pol["W_bf16"], pol["b"], "bf16", wl.sigma_action, 0, n)
    critic = B.Policy(cw["dims"], cw["W_bf16"], cw["b"], "bf16", 1.0, 0, n)
    if staged:
        g_env.attach_policy(actor)
    # oracle pass: fixes the simulator states of every step
    obs_o = [o_env.reset_all(0)]
    sims, reward_o, flags_o = {}, [], []
    for t in range(T):
        s = 1 + t
        sim = W.synth_sim_state(sc.skel, sc.lib, o_env.clip_id, o_env.t.astype(np.float64) + wl.dt, s, wl)
        sims[s] = torch.from_numpy(np.ascontiguousarray(sim)).cuda()
        out = o_env.step(s, sim, want_terms=False)
        obs_o.append(out["obs"]); reward_o.append(out["reward"]); flags_o.append(out["flags"])
    st = R.RolloutStorage(T, n, pol["dims"][-1], ld, keep_obs=True)
    g_env.reset_all(st.obs_row(0), 0)
    R.collect(g_env, actor, critic, st, lambda s: sims[s], 1, gamma, lam, True, staged=staged)
    torch.cuda.synchronize()
    assert g_env.device_status() == 0 and actor.device_status() == 0 and critic.device_status() == 0
    flags = st.flags.cpu().numpy()
    np.testing.assert_array_equal(flags, np.stack(flags_o))
    assert (flags != 0).any()                                     # h_min = 0.8 ends some episodes
    assert_close(st.reward.cpu().numpy(), np.stack(reward_o), what="stored rewards")
    for t in range(T + 1):
        got = st.obs[t, :, :wl.obs_dim].cpu().numpy()
        assert np.abs(got - obs_o[t]).max() < 1e-3                # loose here; the env parity tests hold the real bar
    for t in (0, T - 1):
        want = O.policy_forward(pol["dims"], pol["W"], pol["b"], wl.sigma_action, 0, 1 + t, obs_o[t],
                                bf16_operands=True)
        assert_mean_close(st.mean[t].cpu().numpy(), want["mean"], 2e-2, "stored means")
        assert_close(st.logp[t].cpu().numpy(), want["logp"], atol=1e-3, rtol=1e-5, what="stored logp")
        assert_close((st.action[t] - st.mean[t]).cpu().numpy(), wl.sigma_action * want["z"], atol=1e-5, rtol=1e-4,
                     what="stored action noise")
    for t in (0, T):
        want = O.policy_forward(cw["dims"], cw["W"], cw["b"], 1.0, 0, 0, obs_o[t], bf16_operands=True)["mean"]
        assert_mean_close(st.value[t].cpu().numpy()[:, None], want, 2e-2, "stored values")
    reward, value = st.reward.cpu().numpy(), st.value.cpu().numpy()
    adv_o, ret_o = O.gae(reward, value, flags, gamma, lam, True)
    tol = gae_tolerance(T, gamma, lam, reward, value, adv_o)
    assert np.abs(st.advantage.cpu().numpy() - adv_o).max() <= tol
    assert np.abs(st.returns.cpu().numpy() - ret_o).max() <= tol
    g_env.attach_policy(None)


@pytest.mark.parametrize("staged", [False, True], ids=["fp32-rows", "staged-bf16-rows"])
def test_collect_with_the_extended_observation_feeds_actions_back(staged):
    """With the observation extension on, the policy's input row is wider (further end-effector frames,
    previous action) and every step's actions show up in the next row, zeroed where the env was reset."""
    from paper_2609_09821_b200 import rollout as R
    wl = W.WORKLOADS["cfg3_16384_lib32"]
    sc = Scene(wl)
    n, T, A, F = 256, 4, wl.act_dim, 2
    D = wl.obs_dim + (F - 1) * 9 * sc.o_skel.n_ee + A
    ld = B.padded_ld(D)
    dims = (D, 128, A)
    pw = W.make_policy_weights(dims, "bf16", 3)
    g_env = B.Env(sc.g_skel, sc.g_clips, B.make_env_config(n, wl.dt, 0, W.REWARD_MULT, 0.8, ld))
    st = R.RolloutStorage(T, n, A, ld, keep_obs=True)
    assert g_env.set_obs_extension(F, st.action[0]) == D
    actor = B.Policy(dims, pw["W_bf16"], pw["b"], "bf16", 0.1, 0, n)
    if staged:
        g_env.attach_policy(actor)
    g_env.reset_all(st.obs_row(0), 0)
    c, t, _ = g_env.get_state()
    sims = {s: W.synth_sim_state_torch(sc.skel, sc.lib, c.long(), t.double() + wl.dt * s, s, wl) for s in range(1, T + 1)}
    R.collect(g_env, actor, None, st, lambda s: sims[s], 1, 0.99, 0.95, staged=staged)
    torch.cuda.synchronize()
    assert g_env.device_status() == 0 and actor.device_status() == 0
    assert not st.obs[0, :, D - A:D].any()
    some_reset = False
    for k in range(T):
        reset = st.flags[k] != 0
        some_reset |= bool(reset.any())
        tail = st.obs[k + 1, :, D - A:D]
        assert torch.equal(tail[~reset], st.action[k][~reset]) and not tail[reset].any()
        assert bool((st.obs[k + 1, :, D:] == 0).all())
    assert some_reset
    # the policy read the whole extended row: its means match the oracle's on the stored rows
    want = O.policy_forward(dims, pw["W"], pw["b"], 0.1, 0, T, st.obs[T - 1].cpu().numpy().astype(np.float64),
                            bf16_operands=True)
    assert_mean_close(st.mean[T - 1].cpu().numpy(), want["mean"], 2e-2, "means on extended rows")
    g_env.attach_policy(None)


# ---------------------------------------------------------------- per-dimension standard deviation
@pytest.mark.parametrize("dtype,dims", [("f32", (361, 64, 28)), ("bf16", (361, 128, 28)), ("bf16", (577, 256, 69))])
def test_per_dimension_log_std(dtype, dims):
    from tests.parity import assert_close
    n, seed, step = 500, 0xABCDEF12345, 7
    pw = W.make_policy_weights(dims, dtype, 3)
    A = dims[-1]
    g = np.random.default_rng(5)
    obs = g.standard_normal((n, dims[0])).astype(np.float32)
    log_std = g.uniform(-2.5, 0.5, A).astype(np.float32)          # around the paper's initial values (-2.0, -1.5)
    pol = B.Policy(dims, pw["W_bf16"] if dtype == "bf16" else pw["W"], pw["b"], dtype, 0.1, seed, n)
    ld = B.padded_ld(dims[0])
    obs_g = torch.zeros((n, ld), device="cuda")
    obs_g[:, :dims[0]] = torch.from_numpy(obs).cuda()
    mean, act, logp = (torch.empty((n, A), device="cuda"), torch.empty((n, A), device="cuda"), torch.empty(n, device="cuda"))
    pol.set_log_std(torch.from_numpy(log_std).cuda())
    pol.forward(step, obs_g, mean, act, logp)
    torch.cuda.synchronize()
    want = O.policy_forward(dims, pw["W"], pw["b"], 0.1, seed, step, obs.astype(np.float64),
                            bf16_operands=dtype == "bf16", log_std=log_std)
    assert_mean_close(mean.cpu().numpy(), want["mean"], 2e-2 if dtype == "bf16" else 1e-4, "means")
    noise = (act - mean).cpu().numpy().astype(np.float64)
    assert_close(noise, np.exp(log_std.astype(np.float64)) * want["z"], atol=1e-5, rtol=1e-4, what="per-dimension noise")
    assert_close(logp.cpu().numpy(), want["logp"], atol=1e-3, rtol=1e-5, what="logp")
    # back to the scalar sigma
    pol.set_log_std(None)
    pol.forward(step, obs_g, mean, act, logp)
    torch.cuda.synchronize()
    assert_close((act - mean).cpu().numpy(), 0.1 * want["z"], atol=1e-5, rtol=1e-4, what="scalar noise")
    with pytest.raises(ValueError):
        pol.set_log_std(torch.zeros(A + 1, device="cuda"))
