"""GPU parity: the CUDA library against the CPU oracle on the same seeded inputs,
through the C ABI.  Small cases span several 32-env tiles plus a ragged tail;
full-size cases run the launch configuration the benchmark times."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2609_09821_b200 import binding as B
from paper_2609_09821_b200 import workloads as W
from tests.parity import Pair, Scene, assert_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def scenes():
    cache = {}

    def get(name):
        if name not in cache:
            cache[name] = Scene(W.WORKLOADS[name])
        return cache[name]
    return get


def test_library_is_loaded_and_launches_kernels(scenes):
    before = B.launch_count()
    p = Pair(scenes("cfg1_tiny64"), 64)
    p.rollout(steps=1)
    assert B.launch_count() >= before + 2 + 4


# ---------------------------------------------------------------- the five configurations
def test_cfg1_tiny_fp32_full(scenes):
    p = Pair(scenes("cfg1_tiny64"), 64)
    p.rollout()                                   # 10 steps, every env, fp32 policy


@pytest.mark.parametrize("reward", [W.REWARD_FIG5, W.REWARD_ADD4], ids=["fig5", "add4"])
def test_cfg1_additive_rewards(scenes, reward):
    p = Pair(scenes("cfg1_tiny64"), 64, reward=reward, with_policy=False)
    h = p.rollout(steps=4)
    assert np.mean([x["reward"].mean() for x in h]) > 0.01      # not a vacuous all-zero comparison


@pytest.mark.parametrize("n", [1, 31, 33, 77, 1000])
def test_ragged_batches(scenes, n):
    p = Pair(scenes("cfg2_4096"), n)
    p.rollout(steps=3)


@pytest.mark.parametrize("name,n", [("cfg2_4096", 1000), ("cfg4_65536_smpl24", 700), ("cfg5_reset_heavy", 257)])
def test_cta_pair_gemm_on_small_batches(scenes, name, n):
    """The cta_group::2 kernel (normally chosen only for many tiles) forced on a ragged small batch."""
    p = Pair(scenes(name), n, policy_impl=2)
    p.rollout(steps=2)


def test_simt_layers_with_bf16_weights(scenes):
    """The SIMT cross-check path (bf16 weights, fp32 activations) against the unrounded oracle."""
    p = Pair(scenes("cfg2_4096"), 200, policy_impl=1)
    p.rollout(steps=2)


def test_cfg2_reduced(scenes):
    p = Pair(scenes("cfg2_4096"), 1024 + 17)
    p.rollout(steps=6)


def test_cfg3_library_reduced(scenes):
    p = Pair(scenes("cfg3_16384_lib32"), 2048 + 5, with_policy=False)
    h = p.rollout(steps=8)
    assert len({int(c) for c in p.o_env.clip_id}) > 16            # many clips in play


def test_cfg4_smpl_reduced(scenes):
    p = Pair(scenes("cfg4_65536_smpl24"), 640 + 3)
    p.rollout(steps=4)


def test_cfg5_reset_heavy_reduced(scenes):
    p = Pair(scenes("cfg5_reset_heavy"), 2048 + 9, write_back=True)
    h = p.rollout(steps=10, policy_every=5)
    rate = np.mean([(x["flags"] != 0).mean() for x in h])
    assert 0.08 < rate < 0.4


@pytest.mark.parametrize("seed", [1, 2])
def test_other_seeds(scenes, seed):
    wl = W.WORKLOADS["cfg3_16384_lib32"]
    p = Pair(scenes("cfg3_16384_lib32"), 512, seed=seed, with_policy=False)
    p.rollout(steps=4)


@pytest.mark.parametrize("name", ["cfg2_4096", "cfg3_16384_lib32", "cfg4_65536_smpl24", "cfg5_reset_heavy"])
def test_full_size(scenes, name):
    """Full env count in the benchmark's launch configuration; every env's observation, reward,
    flags and state against the oracle, the policy on a sample of envs."""
    wl = W.WORKLOADS[name]
    p = Pair(scenes(name), wl.n_envs, policy_sample=192, want_terms=False)
    p.rollout(steps=3, device="cuda")
    print("%s: largest observation error %.2e, largest reward error %.2e" % (name, p.max_err["obs"], p.max_err["reward"]))


@pytest.mark.parametrize("name", ["cfg2_4096", "cfg3_16384_lib32", "cfg4_65536_smpl24", "cfg5_reset_heavy"])
def test_full_batch_policy_step(scenes, name):
    """One policy step on the whole batch of each bf16 configuration: every mean, noise and log-probability
    element against the oracle (every row and column tile of the GEMM chain, CTA pairs included)."""
    wl = W.WORKLOADS[name]
    p = Pair(scenes(name), wl.n_envs, with_policy=True, want_terms=False)
    p.reset_all()
    p.policy_step(1)


@pytest.mark.parametrize("name,n", [("cfg2_4096", 96 + 3), ("cfg3_16384_lib32", 128 + 5), ("cfg4_65536_smpl24", 64 + 7),
                                    ("cfg5_reset_heavy", 256 + 1)])
def test_rollouts_of_the_stated_length(scenes, name, n):
    """Every configuration run to the rollout length it states (32 steps, 64 for the reset-heavy one) on a reduced
    env count: resets, truncations at clip ends and re-draws accumulate over the whole horizon."""
    wl = W.WORKLOADS[name]
    p = Pair(scenes(name), n, write_back=name == "cfg5_reset_heavy")
    h = p.rollout(steps=wl.steps, policy_every=8)
    assert len(h) == wl.steps == (64 if name == "cfg5_reset_heavy" else 32)
    if name == "cfg5_reset_heavy":
        rate = np.mean([(x["flags"] != 0).mean() for x in h])
        assert 0.08 < rate < 0.4


# ---------------------------------------------------------------- edge cases
def test_reward_threshold_termination(scenes):
    """Figure 5's done rule (root height or reward below a threshold); the reward threshold is set
    near the median reward of this workload so that both outcomes occur."""
    p = Pair(scenes("cfg1_tiny64"), 64, reward=W.REWARD_FIG5, h_min=0.55, r_min=0.865, with_policy=False)
    h = p.rollout(steps=5)
    frac = np.mean([(x["flags"] & 1).mean() for x in h])
    assert 0.05 < frac < 0.95


def test_all_reset_and_none_reset(scenes):
    for h_min in (10.0, -10.0):
        p = Pair(scenes("cfg1_tiny64"), 64, h_min=h_min, with_policy=False, write_back=True)
        h = p.rollout(steps=3)
        assert all(((x["flags"] & 1) == (1 if h_min > 0 else 0)).all() for x in h)


def test_min_ld_obs_and_padded_component_stride(scenes):
    p = Pair(scenes("cfg1_tiny64"), 50, ld_obs=364, stride_pad=14, with_policy=False)
    p.rollout(steps=3)


def test_single_body_and_max_bodies():
    for J in (1, 2, 32):
        wl = W.Workload("edge_J%d" % J, 40, "custom", 2, (5, 9), 3, (24 * J + 1, 64, 8), "f32")
        rng = np.random.default_rng(J)
        parents = np.array([-1] + [int(rng.integers(max(0, j - 3), j)) for j in range(1, J)], np.int32)
        if J == 32:
            parents = np.arange(-1, 31, dtype=np.int32)           # one 32-link chain: deepest possible
        offsets = rng.uniform(-0.3, 0.3, (J, 3)).astype(np.float32)
        offsets[0] = 0
        has_child = np.zeros(J, bool)
        has_child[parents[1:]] = True
        skel = dict(kind="custom", J=J, parents=parents, offsets=offsets,
                    masses=rng.uniform(1, 3, J).astype(np.float32), ee_ids=np.nonzero(~has_child)[0].astype(np.int32))
        lib = W.make_clip_library(J, 2, (5, 9), 30.0, seed=J)
        pol = W.make_policy_weights(wl.mlp_dims, "f32", seed=J)
        p = Pair(Scene(wl, skel, lib, pol), 40)
        p.rollout(steps=3)
        print("J = %d: largest observation error %.2e" % (J, p.max_err["obs"]))


def test_sharded_envs_reproduce_the_unsplit_batch(scenes):
    sc = scenes("cfg5_reset_heavy")
    whole = Pair(sc, 96, with_policy=True)
    whole.reset_all()
    obs_whole = whole.obs_g.clone()
    parts = [Pair(sc, 48, env_base=0), Pair(sc, 48, env_base=48)]
    for q in parts:
        q.reset_all()
    assert torch.equal(torch.cat([q.obs_g for q in parts]), obs_whole)
    sim = W.synth_sim_state_torch(sc.skel, sc.lib, torch.from_numpy(whole.o_env.clip_id.astype(np.int64)),
                                  torch.from_numpy(whole.o_env.t.astype(np.float64)) + sc.wl.dt, 1, sc.wl)
    whole.policy_step(1)
    whole.env_step(1, sim)
    for k, q in enumerate(parts):
        q.policy_step(1)
        q.env_step(1, sim[:, 48 * k:48 * (k + 1)].contiguous())
    assert torch.equal(torch.cat([q.obs_g for q in parts]), whole.obs_g)
    assert torch.equal(torch.cat([q.action_g for q in parts]), whole.action_g)
    assert torch.equal(torch.cat([q.flags_g for q in parts]), whole.flags_g)


def test_deterministic_and_resumable(scenes):
    sc = scenes("cfg5_reset_heavy")
    a = Pair(sc, 300, with_policy=False)
    hist = []
    sims = []
    a.reset_all()

    def consume(s, sim):
        sims.append(sim)
        a.env_step(s, sim)
        hist.append((a.obs_g.clone(), a.reward_g.clone(), a.flags_g.clone(), a.g_env.get_state()))

    W.rollout_inputs(sc.wl, sc.skel, sc.lib, lambda: (a.o_env.clip_id, a.o_env.t), consume, steps=6)
    # second env resumes at step 4 from the saved state and must reproduce steps 4..6 bit for bit
    b = B.Env(sc.g_skel, sc.g_clips, B.make_env_config(300, sc.wl.dt, sc.wl.seed, W.REWARD_MULT, sc.wl.h_min,
                                                       a.ld_obs))
    c, t, l = hist[2][3]
    b.set_state(c, t, l)
    obs = b.new_obs()
    rew = torch.empty(300, device="cuda")
    fl = torch.empty(300, dtype=torch.uint8, device="cuda")
    for s in (4, 5, 6):
        b.step(s, sims[s - 1].cuda(), obs, rew, fl)
        torch.cuda.synchronize()
        assert torch.equal(obs, hist[s - 1][0]) and torch.equal(rew, hist[s - 1][1]) and torch.equal(fl, hist[s - 1][2])


def test_steps_are_capturable_and_replay_bit_exact(scenes):
    """Per-step calls only enqueue work: a CUDA graph of a whole rollout replays to the same bits."""
    sc = scenes("cfg2_4096")
    n, steps = 600, 5
    p = Pair(sc, n)
    p.g_env.attach_policy(p.policy)
    p.reset_all()
    c0, t0, l0 = p.g_env.get_state()
    obs0 = p.obs_g.clone()
    sims = []

    def consume(s, sim):
        sims.append(sim.cuda())
        p.policy.forward_staged(s, n, p.mean_g, p.action_g, p.logp_g)
        p.env_step(s, sim)

    W.rollout_inputs(sc.wl, sc.skel, sc.lib, lambda: (p.o_env.clip_id, p.o_env.t), consume, steps=steps)
    want = (p.obs_g.clone(), p.reward_g.clone(), p.flags_g.clone(), p.action_g.clone(), p.g_env.get_state())
    # same rollout again as one captured graph, from the same initial state
    stream = p.g_env.stream
    p.g_env.set_state(c0, t0, l0)
    p.g_env.reset_all(p.obs_g, 0)            # refills the policy's staged input as well
    assert torch.equal(p.obs_g, obs0)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    env2 = B.Env(sc.g_skel, sc.g_clips, B.make_env_config(n, sc.wl.dt, sc.wl.seed, W.REWARD_MULT, sc.wl.h_min, p.ld_obs),
                 stream=side)
    pol2 = B.Policy(sc.pol["dims"], sc.pol["W_bf16"], sc.pol["b"], "bf16", sc.wl.sigma_action, sc.wl.seed, n, stream=side)
    env2.attach_policy(pol2)
    obs = env2.new_obs()
    rew = torch.empty(n, device="cuda")
    fl = torch.empty(n, dtype=torch.uint8, device="cuda")
    mean = torch.empty((n, p.A), device="cuda")
    act = torch.empty((n, p.A), device="cuda")
    with torch.cuda.stream(side):
        env2.reset_all(obs, 0)
    side.synchronize()
    with torch.cuda.graph(g, stream=side):
        for s in range(1, steps + 1):
            pol2.forward_staged(s, n, mean, act)
            env2.step(s, sims[s - 1], obs, rew, fl)
    for _ in range(2):                        # replaying twice from the same state gives the same result
        env2.set_state(c0, t0, l0)
        with torch.cuda.stream(side):
            env2.reset_all(obs, 0)
        side.synchronize()
        g.replay()
        torch.cuda.synchronize()
        c, t, l = env2.get_state()
        assert torch.equal(obs, want[0]) and torch.equal(rew, want[1]) and torch.equal(fl, want[2])
        assert torch.equal(act, want[3])
        assert torch.equal(c, want[4][0]) and torch.equal(t, want[4][1]) and torch.equal(l, want[4][2])


def test_bad_simulated_quaternion_sets_status_not_a_fault(scenes):
    sc = scenes("cfg1_tiny64")
    p = Pair(sc, 64, with_policy=False)
    p.reset_all()
    sim = W.synth_sim_state_torch(sc.skel, sc.lib, torch.from_numpy(p.o_env.clip_id.astype(np.int64)),
                                  torch.from_numpy(p.o_env.t.astype(np.float64)) + sc.wl.dt, 1, sc.wl).cuda()
    sim[3 * 15 + 4 * 3:3 * 15 + 4 * 3 + 4, 5] = 0.0            # body 3 of env 5: zero quaternion
    sim[3 * 15 + 4 * 7, 9] = float("nan")
    p.g_env.step(1, sim, p.obs_g, p.reward_g, p.flags_g, None)
    assert p.g_env.device_status() & 1
    ok = np.ones(64, bool)
    ok[[5, 9]] = False
    assert torch.isfinite(p.obs_g[torch.from_numpy(ok).cuda()]).all()
    assert torch.isfinite(p.obs_g[5]).all()


@pytest.mark.parametrize("n", [500, 49280], ids=["one-upload", "four-env-ranges"])
def test_host_buffer_step_matches_device_step(scenes, n):
    """From 49152 envs on the upload and the env kernel are split into four env ranges; same results."""
    sc = scenes("cfg2_4096")
    p = Pair(sc, n, policy_sample=300)
    p.reset_all()
    env2 = B.Env(sc.g_skel, sc.g_clips, B.make_env_config(n, sc.wl.dt, sc.wl.seed, W.REWARD_MULT, sc.wl.h_min, p.ld_obs))
    env2.reset_all_host(0)
    act = torch.empty((n, p.A)).pin_memory()
    rew = torch.empty(n).pin_memory()
    fl = torch.empty(n, dtype=torch.uint8).pin_memory()
    for s in (1, 2):
        sim = W.synth_sim_state_torch(sc.skel, sc.lib, torch.from_numpy(p.o_env.clip_id.astype(np.int64)),
                                      torch.from_numpy(p.o_env.t.astype(np.float64)) + sc.wl.dt, s, sc.wl)
        p.policy_step(s)
        p.env_step(s, sim)
        B.step_host(env2, p.policy, s, sim.contiguous().pin_memory(), act, rew, fl)
        assert torch.equal(act, p.action_g.cpu()) and torch.equal(rew, p.reward_g.cpu()) and torch.equal(fl, p.flags_g.cpu())


def test_staged_policy_input_matches_the_conversion_pass(scenes):
    """An env attached to a tensor-core policy leaves bf16 observation rows in the policy's input
    buffer; the policy run on them must equal the policy run on the fp32 rows bit for bit."""
    sc = scenes("cfg4_65536_smpl24")
    n = 700
    p = Pair(sc, n)
    p.g_env.attach_policy(p.policy)
    p.reset_all()
    mean2 = torch.empty_like(p.mean_g)
    act2 = torch.empty_like(p.action_g)
    logp2 = torch.empty_like(p.logp_g)
    for s in (1, 2, 3):
        p.policy_step(s)                                              # fp32 rows through the conversion pass
        p.policy.forward_staged(s, n, mean2, act2, logp2)              # bf16 rows written by the env kernel
        torch.cuda.synchronize()
        assert torch.equal(mean2, p.mean_g) and torch.equal(act2, p.action_g) and torch.equal(logp2, p.logp_g)
        sim = W.synth_sim_state_torch(sc.skel, sc.lib, torch.from_numpy(p.o_env.clip_id.astype(np.int64)),
                                      torch.from_numpy(p.o_env.t.astype(np.float64)) + sc.wl.dt, s, sc.wl)
        p.env_step(s, sim)
    p.g_env.attach_policy(None)


def test_bf16_rows_only_when_the_fp32_observation_is_not_asked_for(scenes):
    """With a policy attached obs_out may be NULL: the staged bf16 rows (and everything else the step returns)
    are the same bits as with the fp32 rows written as well; without a policy NULL is an error."""
    sc = scenes("cfg3_16384_lib32")
    wl, n = sc.wl, 1000
    ld = B.padded_ld(wl.obs_dim)
    pol = sc.pol
    outs = []
    for with_obs in (True, False):
        env = B.Env(sc.g_skel, sc.g_clips, B.make_env_config(n, wl.dt, 3, W.REWARD_MULT, 0.8, ld))
        policy = B.Policy(pol["dims"], pol["W_bf16"], pol["b"], "bf16", wl.sigma_action, 3, n)
        env.attach_policy(policy)
        obs = torch.zeros((n, ld), device="cuda") if with_obs else None
        rew, fl = torch.empty(n, device="cuda"), torch.empty(n, dtype=torch.uint8, device="cuda")
        mean, act, logp = torch.empty((n, wl.act_dim), device="cuda"), torch.empty((n, wl.act_dim), device="cuda"), torch.empty(n, device="cuda")
        env.reset_all(obs, 0)
        hist = []
        for s in range(1, 4):
            c, t, _ = env.get_state()
            sim = W.synth_sim_state_torch(sc.skel, sc.lib, c.long(), t.double() + wl.dt, s, wl)
            policy.forward_staged(s, n, mean, act, logp)
            env.step(s, sim, obs, rew, fl)
            hist.append((mean.clone(), act.clone(), rew.clone(), fl.clone()))
        outs.append(hist)
        env.attach_policy(None)
        if not with_obs:
            with pytest.raises(B.ImError):
                env.step(4, sim, None, rew, fl)              # detached: the fp32 rows are the only output
    for a, b in zip(*outs):
        for x, y in zip(a, b):
            assert torch.equal(x, y)
    assert bool((outs[0][-1][3] != 0).any())


def test_reset_draws_bit_exact_over_many_counters(scenes):
    sc = scenes("cfg3_16384_lib32")
    n = 100000
    p = Pair(sc, n, seed=0xDEADBEEFCAFE, with_policy=False)
    p.o_env.reset_all(0)
    obs = torch.empty((n, p.ld_obs), device="cuda")
    p.g_env.reset_all(obs, 0)
    p.check_state("100k resets")


def test_invalid_arguments_are_rejected(scenes):
    sc = scenes("cfg1_tiny64")
    with pytest.raises(B.ImError):
        B.Env(sc.g_skel, sc.g_clips, B.make_env_config(64, sc.wl.dt, 0, W.REWARD_MULT, 0.3, 360))     # ld_obs < D
    with pytest.raises(B.ImError):
        B.Env(sc.g_skel, sc.g_clips, B.make_env_config(64, 100.0, 0, W.REWARD_MULT, 0.3, 384))        # dt > clip
    env = B.Env(sc.g_skel, sc.g_clips, B.make_env_config(64, sc.wl.dt, 0, W.REWARD_MULT, 0.3, 384))
    obs = torch.empty((64, 384), device="cuda")
    sim = torch.zeros((13 * 15, 60), device="cuda")                                                   # stride < N
    with pytest.raises(B.ImError):
        env.step(1, sim, obs, torch.empty(64, device="cuda"), torch.empty(64, dtype=torch.uint8, device="cuda"))
