"""GPU parity on shapes and settings off the benchmark configurations: odd policy widths and
depths, control intervals that do not match the keyframe rate, clips of different rates and of
the minimum length, explicit end-effectors, uniform masses, zero reward weights."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2609_09821_b200 import binding as B
from paper_2609_09821_b200 import workloads as W
from tests.parity import Pair, Scene

pytestmark = pytest.mark.gpu


def _scene(name, mlp_dims, mlp_dtype="bf16", skeleton="humanoid15", n_clips=3, frames=(20, 40), dt=1.0 / 30.0,
           fps=None, seed=5, masses=True, ee_ids=None, **kw):
    wl = W.Workload(name, 256, skeleton, n_clips, frames, 4, tuple(mlp_dims), mlp_dtype, dt=dt, seed=seed, **kw)
    skel = W.make_skeleton(skeleton, seed)
    lib = W.make_clip_library(skel["J"], n_clips, frames, 30.0, seed)
    if fps is not None:
        lib["fps"] = np.asarray(fps, np.float32)
    pol = W.make_policy_weights(mlp_dims, mlp_dtype, seed)
    sc = Scene.__new__(Scene)
    sc.wl, sc.skel, sc.lib, sc.pol, sc.J = wl, skel, lib, pol, skel["J"]
    m = skel["masses"] if masses else None
    sc.o_skel = O.Skeleton(skel["parents"], skel["offsets"], m, ee_ids)
    sc.o_clips = O.Clips(sc.o_skel, lib["n_frames"], lib["fps"], lib["root_pos"], lib["local_quat"])
    sc.g_skel = B.Skeleton(skel["parents"], skel["offsets"], m, ee_ids)
    sc.g_clips = B.Clips(sc.g_skel, lib["n_frames"], lib["fps"], lib["root_pos"], lib["local_quat"])
    return sc


@pytest.mark.parametrize("dims", [
    (361, 64, 28),                       # one narrow hidden layer: 64-column tiles
    (361, 128, 192, 8),                  # 128- and 64-column tiles
    (361, 256, 64, 64, 64, 64, 64, 5),   # seven layers
    (361, 512, 80),                      # widest action the Gaussian head takes
    (361, 1024, 1),                      # a single output
], ids=lambda d: "x".join(map(str, d)))
def test_policy_shapes_on_the_tensor_path(dims):
    sc = _scene("edge_policy", dims)
    p = Pair(sc, 300)
    p.rollout(steps=2)


def test_unsupported_policy_shapes_are_rejected():
    pol = W.make_policy_weights((361, 100, 28), "bf16", 0)           # hidden width not a multiple of 64
    with pytest.raises(B.ImError) as e:
        B.Policy(pol["dims"], pol["W_bf16"], pol["b"], "bf16", 0.1, 0, 64)
    assert e.value.status == -6
    pol = W.make_policy_weights((361, 128, 96), "bf16", 0)           # action wider than the head's staging
    with pytest.raises(B.ImError) as e:
        B.Policy(pol["dims"], pol["W_bf16"], pol["b"], "bf16", 0.1, 0, 64)
    assert e.value.status == -6
    pol = W.make_policy_weights((361, 28), "bf16", 0)                # a single layer has no hidden GEMM
    with pytest.raises(B.ImError) as e:
        B.Policy(pol["dims"], pol["W_bf16"], pol["b"], "bf16", 0.1, 0, 64)
    assert e.value.status == -6


@pytest.mark.parametrize("dt", [1.0 / 60.0, 0.05, 1.0 / 30.0 + 1e-4])
def test_control_interval_off_the_keyframe_rate(dt):
    sc = _scene("edge_dt", (361, 64, 28), "f32", dt=dt)
    p = Pair(sc, 200, with_policy=False)
    p.rollout(steps=6)


def test_clips_of_different_rates():
    sc = _scene("edge_fps", (361, 64, 28), "f32", n_clips=4, frames=(12, 30), fps=[24.0, 30.0, 60.0, 120.0],
                dt=1.0 / 120.0)
    # the 120 frames-per-second clip carries velocities four times the benchmark's: see Pair.vel_ulps
    p = Pair(sc, 200, with_policy=False, vel_ulps=4)
    h = p.rollout(steps=8)
    assert any((x["flags"] & 2).any() for x in h)        # the short, fast clips truncate within a few steps


def test_two_keyframe_clips_reset_every_step():
    sc = _scene("edge_k2", (361, 64, 28), "f32", n_clips=2, frames=(2, 2))
    p = Pair(sc, 100, with_policy=False)
    h = p.rollout(steps=3)
    assert all((x["flags"] & 2).all() for x in h)        # D = dt: the next step would always pass the end
    assert np.all(p.o_env.t == 0.0)


def test_uniform_masses_explicit_end_effectors_and_zero_weights():
    zero = dict(mode=0, a=[0.0] * 7, w=[0.0] * 7)
    sc = _scene("edge_skel", (361, 64, 28), "f32", masses=False, ee_ids=[3, 6, 9])
    p = Pair(sc, 150, reward=zero, with_policy=False)
    h = p.rollout(steps=2)
    assert all(np.all(x["reward"] == 1.0) for x in h)     # exp(-0) exactly
    p = Pair(sc, 150, reward=W.REWARD_ADD4, with_policy=False)
    p.rollout(steps=2)


def test_smpl_skeleton_with_fp32_policy():
    sc = _scene("edge_smpl_f32", (577, 96, 40, 69), "f32", skeleton="smpl24")
    p = Pair(sc, 130)
    p.rollout(steps=2)


def test_zero_envs_is_an_error():
    sc = _scene("edge_zero", (361, 64, 28), "f32")
    with pytest.raises(B.ImError):
        B.Env(sc.g_skel, sc.g_clips, B.make_env_config(0, 1 / 30, 0, W.REWARD_MULT, 0.3, 384))


# ---------------------------------------------------------------- optional env semantics
@pytest.mark.parametrize("skeleton,dims", [("humanoid15", (361, 64, 28)), ("smpl24", (577, 64, 69))])
def test_motion_randomisation_of_reset_states(skeleton, dims):
    """Reset envs start from the randomised reference state: observation and written-back body
    states against the oracle, with terminations frequent enough that many envs reset each step."""
    sc = _scene("edge_noise_" + skeleton, dims, "f32", skeleton=skeleton, sigma_root=0.05)
    p = Pair(sc, 300, h_min=W.ROOT_HEIGHT, write_back=True, with_policy=False, reset_noise_std=0.05, seed=77)
    h = p.rollout(steps=6)
    frac = np.mean([(x["flags"] != 0).mean() for x in h])
    assert 0.2 < frac < 0.9                                # resets and survivors both well represented
    # the randomisation is there: the same rollout without it observes different reset states
    q = Pair(sc, 300, h_min=W.ROOT_HEIGHT, write_back=True, with_policy=False, seed=77)
    q.reset_all()
    p2 = Pair(sc, 300, h_min=W.ROOT_HEIGHT, write_back=True, with_policy=False, reset_noise_std=0.05, seed=77)
    p2.reset_all()
    assert np.abs(p2.obs_o - q.obs_o).max() > 1e-2


def test_grace_steps_hold_off_termination():
    sc = _scene("edge_grace", (361, 64, 28), "f32", n_clips=2, frames=(12, 14))
    p = Pair(sc, 200, h_min=10.0, with_policy=False, grace_steps=3)          # h_min 10: the height test always fires
    h = p.rollout(steps=12)
    term = np.array([(x["flags"] & 1) for x in h])
    trunc = np.array([(x["flags"] >> 1) for x in h])
    assert not term[:3].any() and term[3:].any()           # nothing terminates in the first three steps
    assert trunc.any()                                     # the 11- to 13-interval clips still truncate
    _, _, ep = p.g_env.get_state()
    assert int(ep.max()) <= 3


def test_env_options_are_validated():
    sc = _scene("edge_opts", (361, 64, 28), "f32")
    for kw in (dict(grace_steps=-1), dict(reset_noise_std=-0.1), dict(reset_noise_std=float("nan"))):
        with pytest.raises(B.ImError):
            B.Env(sc.g_skel, sc.g_clips, B.make_env_config(64, 1 / 30, 0, W.REWARD_MULT, 0.3, 384, **kw))


def test_adaptive_initialisation_draws_and_counts_match_the_oracle():
    """Weighted (clip, phase bin) resets: clip ids, start times (bit patterns) and the start/failure
    counts against the oracle over a rollout with frequent terminations; then new weights mid-run."""
    sc = _scene("edge_bins", (361, 64, 28), "f32", n_clips=4, frames=(20, 45), sigma_root=0.05)
    n, B_ = 500, 6
    g = np.random.default_rng(3)
    w = g.uniform(0.0, 1.0, (4, B_)).astype(np.float32)
    w[1, :] = 0.0                                        # a clip that is never started
    w[2, 3] = 0.0
    p = Pair(sc, n, h_min=W.ROOT_HEIGHT, with_policy=False, seed=21, grace_steps=1)
    p.o_env.set_reset_bins(B_, w)
    p.g_env.set_reset_bins(B_, w)
    h = p.rollout(steps=5)                               # Pair checks clip ids and time bit patterns every step
    assert sum(int((x["flags"] & 1).sum()) for x in h) > 200
    starts, failures = p.g_env.reset_stats()
    np.testing.assert_array_equal(starts.cpu().numpy().ravel(), p.o_env.stat_starts.view(np.int32))
    np.testing.assert_array_equal(failures.cpu().numpy().ravel(), p.o_env.stat_failures.view(np.int32))
    assert starts[1].sum() == 0 and starts[2, 3] == 0 and int(starts.sum()) > n
    # new weights, same bin count: tables are replaced, counts go on
    w2 = np.ones((4, B_), np.float32)
    p.o_env.set_reset_bins(B_, w2)
    p.o_env.stat_starts[:] = starts.cpu().numpy().ravel().view(np.uint32)
    p.o_env.stat_failures[:] = failures.cpu().numpy().ravel().view(np.uint32)
    p.g_env.set_reset_bins(B_, w2)
    sim = W.synth_sim_state_torch(sc.skel, sc.lib, torch.from_numpy(p.o_env.clip_id.astype(np.int64)),
                                  torch.from_numpy(p.o_env.t.astype(np.float64)) + sc.wl.dt, 6, sc.wl)
    p.env_step(6, sim)
    starts, failures = p.g_env.reset_stats(clear=True)
    np.testing.assert_array_equal(starts.cpu().numpy().ravel(), p.o_env.stat_starts.view(np.int32))
    np.testing.assert_array_equal(failures.cpu().numpy().ravel(), p.o_env.stat_failures.view(np.int32))
    assert starts[1].sum() > 0
    z, _ = p.g_env.reset_stats()
    assert int(z.sum()) == 0
    # back to the uniform draw
    p.g_env.set_reset_bins(0)
    with pytest.raises(B.ImError):
        p.g_env.reset_stats()
    for bad in (np.zeros((4, B_)), -np.ones((4, B_)), np.full((4, B_), np.nan)):
        with pytest.raises(B.ImError):
            p.g_env.set_reset_bins(B_, bad)


def test_bin_weights_adapted_on_the_device_match_the_oracle():
    """im_env_adapt_reset_bins rebuilds the reset table from the failure counts without leaving the stream:
    after it the weighted draws (clip ids, start-time bit patterns, checked by Pair every step) and the
    restarted counts must keep matching the oracle, eagerly and when the call is replayed from a CUDA graph."""
    sc = _scene("edge_adapt", (361, 64, 28), "f32", n_clips=4, frames=(20, 45), sigma_root=0.05)
    n, B_ = 600, 5
    p = Pair(sc, n, h_min=W.ROOT_HEIGHT, with_policy=False, seed=5)
    w = np.ones((4, B_), np.float32)
    p.o_env.set_reset_bins(B_, w)
    p.g_env.set_reset_bins(B_, w)
    p.reset_all()
    step = [0]

    def advance(k):
        for _ in range(k):
            step[0] += 1
            sim = W.synth_sim_state_torch(sc.skel, sc.lib, torch.from_numpy(p.o_env.clip_id.astype(np.int64)),
                                          torch.from_numpy(p.o_env.t.astype(np.float64)) + sc.wl.dt, step[0], sc.wl)
            p.env_step(step[0], sim)

    advance(4)
    assert int(p.o_env.stat_failures.sum()) > 100
    before = p.o_env.reset_cdf.copy()
    p.o_env.adapt_reset_bins(0.25)
    p.g_env.adapt_reset_bins(0.25)
    assert (p.o_env.reset_cdf != before).any()
    advance(4)                                              # draws from the adapted table, bit for bit
    starts, failures = p.g_env.reset_stats()
    np.testing.assert_array_equal(starts.cpu().numpy().ravel(), p.o_env.stat_starts.view(np.int32))
    np.testing.assert_array_equal(failures.cpu().numpy().ravel(), p.o_env.stat_failures.view(np.int32))
    assert int(starts.sum()) < 4 * n                        # the counts restarted at the adaptation
    # keeping the counts
    p.o_env.adapt_reset_bins(2.0, clear=False)
    p.g_env.adapt_reset_bins(2.0, clear=False)
    advance(3)
    starts, failures = p.g_env.reset_stats()
    np.testing.assert_array_equal(starts.cpu().numpy().ravel(), p.o_env.stat_starts.view(np.int32))
    np.testing.assert_array_equal(failures.cpu().numpy().ravel(), p.o_env.stat_failures.view(np.int32))
    assert p.g_env.device_status() == 0
    # the call is stream-ordered and capturable: a second env on a side stream adapts from a graph replay
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        g2 = B.Env(sc.g_skel, sc.g_clips, B.make_env_config(n, sc.wl.dt, 5, W.REWARD_MULT, W.ROOT_HEIGHT, p.ld_obs), stream=stream)
        g2.set_reset_bins(B_, w)
        obs2 = torch.empty((n, p.ld_obs), device="cuda")
        g2.reset_all(obs2, 0)                               # fills the start counts
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            g2.adapt_reset_bins(3.0, clear=True)
        graph.replay()
        g2.reset_all(obs2, 7)
        stream.synchronize()
        c2, t2, _ = g2.get_state()
        s2, f2 = g2.reset_stats()
    o2 = O.Env(sc.o_skel, sc.o_clips, O.make_env_config(sc.wl.dt, 5, W.REWARD_MULT, W.ROOT_HEIGHT), n)
    o2.set_reset_bins(B_, w)
    o2.reset_all(0)
    o2.adapt_reset_bins(3.0, clear=True)
    o2.reset_all(7)
    np.testing.assert_array_equal(c2.cpu().numpy(), o2.clip_id)
    np.testing.assert_array_equal(t2.cpu().numpy().view(np.uint32), o2.t.view(np.uint32))
    np.testing.assert_array_equal(s2.cpu().numpy().ravel(), o2.stat_starts.view(np.int32))
    assert int(s2.sum()) == n and int(f2.sum()) == 0
    for bad in (0.0, -1.0, float("inf"), float("nan")):
        with pytest.raises(B.ImError):
            p.g_env.adapt_reset_bins(bad)
    p.g_env.set_reset_bins(0)
    with pytest.raises(B.ImError):
        p.g_env.adapt_reset_bins(1.0)


# ---------------------------------------------------------------- simulator-native input arrays
@pytest.mark.parametrize("staged", [False, True], ids=["in_place", "staged"])
@pytest.mark.parametrize("skeleton,dims,n", [("humanoid15", (361, 64, 28), 333), ("smpl24", (577, 64, 69), 200)])
def test_step_on_array_of_structures_inputs(skeleton, dims, n, staged):
    """Body states laid out as a physics engine keeps them -- [env][body][component] with a leading world
    body and angular|linear velocity stored as six floats -- give bit for bit what the component-row
    layout gives (which the other tests hold against the oracle), and reset envs are written back: read in place
    by the env kernel (nothing allocated: the free device memory does not move), or through the staging buffer."""
    sc = _scene("edge_aos_" + skeleton, dims, "f32", skeleton=skeleton, sigma_root=0.05)
    J = sc.J
    p = Pair(sc, n, h_min=W.ROOT_HEIGHT, write_back=True, with_policy=False, seed=9)
    p.reset_all()
    ld = p.ld_obs
    env2 = B.Env(sc.g_skel, sc.g_clips, B.make_env_config(n, sc.wl.dt, 9, W.REWARD_MULT, W.ROOT_HEIGHT, ld,
                                                           write_back_reset=True))
    obs2 = torch.empty((n, ld), device="cuda")
    env2.reset_all(obs2, 0)
    rew2 = torch.empty(n, device="cuda")
    fl2 = torch.empty(n, dtype=torch.uint8, device="cuda")
    terms2 = torch.empty((7, n), device="cuda")
    if staged:
        env2.set_aos_staging(True)
    for s in (1, 2, 3):
        sim = W.synth_sim_state_torch(sc.skel, sc.lib, torch.from_numpy(p.o_env.clip_id.astype(np.int64)),
                                      torch.from_numpy(p.o_env.t.astype(np.float64)) + sc.wl.dt, s, sc.wl).cuda()
        xpos = torch.full((n, J + 1, 3), 7.0, device="cuda")
        xquat = torch.full((n, J + 1, 4), 7.0, device="cuda")
        cvel = torch.full((n, J + 1, 6), 7.0, device="cuda")
        xpos[:, 1:] = sim[0:3 * J].reshape(J, 3, n).permute(2, 0, 1)
        xquat[:, 1:] = sim[3 * J:7 * J].reshape(J, 4, n).permute(2, 0, 1)
        cvel[:, 1:, 3:] = sim[7 * J:10 * J].reshape(J, 3, n).permute(2, 0, 1)
        cvel[:, 1:, :3] = sim[10 * J:13 * J].reshape(J, 3, n).permute(2, 0, 1)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        env2.step_aos(s, xpos[:, 1:], xquat[:, 1:], cvel[:, 1:, 3:], cvel[:, 1:, :3], obs2, rew2, fl2, terms2)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before              # the call itself allocates nothing
        out = p.env_step(s, sim)                                       # component rows, checked against the oracle
        torch.cuda.synchronize()
        assert torch.equal(obs2, p.obs_g) and torch.equal(rew2, p.reward_g) and torch.equal(fl2, p.flags_g)
        assert torch.equal(terms2, p.terms_g)
        reset = torch.from_numpy(out["flags"] != 0).cuda()
        assert 0 < int(reset.sum()) < n
        # reset envs: the reference state arrived in the simulator's arrays; the others and the world body are untouched
        sim_back = torch.cat([xpos[:, 1:].permute(1, 2, 0).reshape(3 * J, n), xquat[:, 1:].permute(1, 2, 0).reshape(4 * J, n),
                              cvel[:, 1:, 3:].permute(1, 2, 0).reshape(3 * J, n),
                              cvel[:, 1:, :3].permute(1, 2, 0).reshape(3 * J, n)])
        assert torch.equal(sim_back[:, ~reset], sim[:, ~reset])
        assert not torch.equal(sim_back[:, reset], sim[:, reset])
        assert (xpos[:, 0] == 7.0).all() and (xquat[:, 0] == 7.0).all() and (cvel[:, 0] == 7.0).all()
        c2, t2, _ = env2.get_state()
        ref = O.reference_state(sc.o_skel, sc.o_clips, int(c2[reset][0]), float(t2[reset][0]))
        e0 = int(torch.nonzero(reset)[0])
        np.testing.assert_allclose(xpos[e0, 1:].cpu().numpy(), ref["p"], atol=1e-5)
        np.testing.assert_allclose(cvel[e0, 1:, :3].cpu().numpy(), ref["w"], atol=1e-4)
    bad = torch.zeros((n, J, 3), device="cuda")
    with pytest.raises(ValueError):
        env2.step_aos(4, bad[:, :, :2], xquat[:, 1:], bad, bad, obs2, rew2, fl2)


@pytest.mark.parametrize("skeleton,dims,n_future,A", [("humanoid15", (361, 64, 28), 3, 28), ("smpl24", (577, 64, 69), 2, 69),
                                                      ("humanoid15", (361, 64, 28), 4, 0), ("smpl24", (577, 64, 69), 1, 5)])
def test_extended_observation_future_frames_and_previous_action(skeleton, dims, n_future, A):
    """End-effector targets of further reference frames and the previous action behind the standard row,
    against the oracle, with resets frequent enough that cleared and copied action entries both occur and with
    clips short enough that future frames run into the clip's end."""
    sc = _scene("edge_ext_" + skeleton, dims, "f32", skeleton=skeleton, n_clips=3, frames=(10, 24), sigma_root=0.05)
    p = Pair(sc, 333, h_min=W.ROOT_HEIGHT, with_policy=False, n_future=n_future, prev_action_dim=A, seed=21)
    assert p.D == 24 * sc.J + 1 + (n_future - 1) * 9 * sc.o_skel.n_ee + A
    h = p.rollout(steps=8)
    frac = np.mean([(x["flags"] != 0).mean() for x in h])
    assert 0.1 < frac < 0.95
    if A:
        tail = p.obs_g[:, p.D - A:p.D].cpu().numpy()
        reset = h[-1]["flags"] != 0
        assert reset.any() and (~reset).any()
        assert not tail[reset].any() and np.array_equal(tail[~reset], p.prev_o[~reset])
    # switching the extension off again restores the standard row
    std = 24 * sc.J + 1
    assert p.g_env.set_obs_extension(1, None) == std
    obs = torch.full((p.n, p.ld_obs), float("nan"), device="cuda")
    p.g_env.reset_all(obs, 0)
    assert bool((obs[:, std:] == 0).all()) and bool(torch.isfinite(obs).all())


def test_all_optional_semantics_together():
    """Grace steps, motion randomisation, weighted initialisation, write-back and the extended observation in one
    env: the options share the kernel's reset and observation phases, so they are also checked in combination."""
    sc = _scene("edge_all_opts", (577, 64, 69), "f32", skeleton="smpl24", n_clips=3, frames=(12, 30), sigma_root=0.05)
    n, B_ = 260, 4
    p = Pair(sc, n, h_min=W.ROOT_HEIGHT, write_back=True, with_policy=False, grace_steps=2, reset_noise_std=0.03,
             n_future=3, prev_action_dim=7, seed=9)
    w = np.random.default_rng(4).uniform(0.1, 1.0, (3, B_)).astype(np.float32)
    p.o_env.set_reset_bins(B_, w)
    p.g_env.set_reset_bins(B_, w)
    h = p.rollout(steps=7)
    flags = np.array([x["flags"] for x in h])
    assert not (flags[:2] & 1).any() and (flags[2:] & 1).any() and (flags >> 1).any()
    starts, failures = p.g_env.reset_stats()
    np.testing.assert_array_equal(starts.cpu().numpy().ravel(), p.o_env.stat_starts.view(np.int32))
    np.testing.assert_array_equal(failures.cpu().numpy().ravel(), p.o_env.stat_failures.view(np.int32))
    assert p.g_env.device_status() == 0


def test_extended_observation_is_validated():
    sc = _scene("edge_ext_bad", (361, 64, 28), "f32")
    env = B.Env(sc.g_skel, sc.g_clips, B.make_env_config(64, 1 / 30, 0, W.REWARD_MULT, 0.3, 384))
    act = torch.zeros((64, 28), device="cuda")
    with pytest.raises(B.ImError):
        env.set_obs_extension(0, None)                       # at least the standard frame
    with pytest.raises(B.ImError):
        env.set_obs_extension(2, act)                        # 361 + 36 + 28 columns do not fit a row stride of 384
    with pytest.raises(ValueError):
        env.set_obs_extension(1, act[:32])                   # fewer rows than envs
    assert env.set_obs_extension(1, act[:, :20]) == 381


# ---------------------------------------------------------------- skeletons with many leaves
def _custom_scene(name, parents, seed, n_clips=2, frames=(6, 12)):
    J = len(parents)
    parents = np.asarray(parents, np.int32)
    wl = W.Workload(name, 100, "custom", n_clips, frames, 3, (24 * J + 1, 64, 8), "f32")
    rng = np.random.default_rng(seed)
    offsets = rng.uniform(-0.3, 0.3, (J, 3)).astype(np.float32)
    offsets[0] = 0
    has_child = np.zeros(J, bool)
    has_child[parents[1:]] = True
    skel = dict(kind="custom", J=J, parents=parents, offsets=offsets, masses=rng.uniform(1, 3, J).astype(np.float32),
                ee_ids=np.nonzero(~has_child)[0].astype(np.int32))
    lib = W.make_clip_library(J, n_clips, frames, 30.0, seed=seed)
    pol = W.make_policy_weights(wl.mlp_dims, "f32", seed=seed)
    return Scene(wl, skel, lib, pol)


WIDE_TREES = {
    "star12": [-1] + [0] * 11,                                     # 11 leaves under the root
    "star32": [-1] + [0] * 31,                                     # 31 leaves: the widest tree there is
    "broom20": [-1, 0, 1, 2] + [3] * 10 + [0] * 6,                 # a 4-link handle with 10 leaves, 6 more at the root
}


@pytest.mark.parametrize("tree", sorted(WIDE_TREES))
@pytest.mark.parametrize("options", ["plain", "resets_written_back", "optional_semantics"])
def test_skeletons_with_more_than_eight_leaves(tree, options):
    """More than 8 root-to-leaf chains make a block of more than 256 threads, which runs the kernel
    instantiation with the smaller register budget: the same comparison with the oracle as everywhere else."""
    sc = _custom_scene("wide_" + tree, WIDE_TREES[tree], seed=len(tree))
    assert (np.bincount(np.asarray(WIDE_TREES[tree][1:]), minlength=len(WIDE_TREES[tree])) == 0).sum() > 8
    if options == "plain":
        p = Pair(sc, 70, with_policy=False)
    elif options == "resets_written_back":
        p = Pair(sc, 70, h_min=W.ROOT_HEIGHT, write_back=True, with_policy=False)
    else:
        p = Pair(sc, 70, h_min=W.ROOT_HEIGHT, write_back=True, with_policy=False, grace_steps=1, reset_noise_std=0.05,
                 n_future=2, prev_action_dim=5)
    h = p.rollout(steps=4)
    if options != "plain":
        assert any((x["flags"] != 0).any() for x in h)


def test_handles_created_from_two_threads_at_once():
    """The one-time kernel set-up (shared-memory opt-in per device) is guarded: two host threads that create their
    first handles of every kind at the same moment both get working ones."""
    import threading
    from paper_2609_09821_b200 import trainer as T
    sc = _scene("edge_threads", (361, 128, 28), "bf16")
    barrier = threading.Barrier(2)
    results, errors = [None, None], []

    def work(i):
        try:
            stream = torch.cuda.Stream()
            barrier.wait()
            with torch.cuda.stream(stream):
                env = B.Env(sc.g_skel, sc.g_clips, B.make_env_config(96, sc.wl.dt, 7, W.REWARD_MULT, 0.3, 384), stream=stream)
                pol = B.Policy(sc.pol["dims"], sc.pol["W_bf16"], sc.pol["b"], "bf16", 0.1, 7, 96, stream=stream)
                tr = T.MlpTrainer(sc.pol["dims"], sc.pol["W"], sc.pol["b"], 128, stream=stream)
                obs = env.new_obs()
                env.reset_all(obs, 0)
                mean, act = torch.empty((96, 28), device="cuda"), torch.empty((96, 28), device="cuda")
                pol.forward(1, obs, mean, act)
                rows = tr.input_rows(128)
                rows.zero_()
                rows[:96, :361] = obs[:, :361].to(torch.bfloat16)
                out = tr.forward(128)[:96].clone()
                stream.synchronize()
                assert env.device_status() == 0 and pol.device_status() == 0 and tr.device_status() == 0
                results[i] = (obs.clone(), mean.clone(), out)
        except Exception as e:                                   # surfaced in the main thread below
            errors.append(e)

    threads = [threading.Thread(target=work, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    for a, b in zip(*results):
        assert torch.equal(a, b)                                 # same seeds, same results from both threads
    assert torch.equal(results[0][1], results[0][2])             # and the trainer's forward is the policy's


def test_training_summaries_accumulate_on_the_device():
    """im_env_set_summary: reward sum (fixed point), terminated / truncated counts and finished-episode lengths
    accumulated by the step kernel itself; counts exact against the oracle's flags and episode lengths, the reward
    sum exact against the kernel's own reward output and within tolerance of the oracle's rewards."""
    sc = _scene("edge_summary", (361, 64, 28), "f32", n_clips=3, frames=(8, 20))
    n = 333
    p = Pair(sc, n, h_min=W.ROOT_HEIGHT, with_policy=False)
    acc = torch.zeros(4, dtype=torch.int64, device="cuda")
    p.g_env.set_summary(acc)
    want = np.zeros(4, np.float64)
    exact_reward = 0
    p.reset_all()
    assert acc.abs().sum().item() == 0                       # the reset-all launch adds nothing
    lens = p.o_env.ep_len.copy()

    def consume(s, sim):
        nonlocal exact_reward, lens
        out = p.env_step(s, sim)
        fl = out["oracle"]["flags"]
        want[0] += out["oracle"]["reward"].sum()
        want[1] += (fl & 1).sum()
        want[2] += ((fl >> 1) & 1).sum()
        want[3] += (lens[fl != 0] + 1).sum()
        exact_reward += int(np.rint(out["reward"].astype(np.float64) * 2.0 ** 40).astype(np.int64).sum())
        lens = p.o_env.ep_len.copy()

    W.rollout_inputs(sc.wl, sc.skel, sc.lib, lambda: (p.o_env.clip_id, p.o_env.t), consume, steps=9)
    got = acc.cpu().numpy()
    assert got[1] == want[1] and got[2] == want[2] and got[3] == want[3]
    assert want[1] > 0 and want[2] > 0 and want[3] > want[1]
    assert int(got[0]) == exact_reward
    assert abs(got[0] / 2.0 ** 40 - want[0]) <= 9 * n * 2e-5
    # detached: later steps leave the accumulator alone
    p.g_env.set_summary(None)
    before = acc.clone()
    sim = W.synth_sim_state_torch(sc.skel, sc.lib, torch.from_numpy(p.o_env.clip_id.astype(np.int64)),
                                  torch.from_numpy(p.o_env.t.astype(np.float64)) + sc.wl.dt, 10, sc.wl)
    p.env_step(10, sim)
    assert torch.equal(acc, before)


# ---------------------------------------------------------------- looped clips
@pytest.mark.parametrize("skeleton,dims,extras", [("humanoid15", (361, 64, 28), dict()),
                                                    ("smpl24", (577, 64, 69), dict(n_future=3, prev_action_dim=4)),
                                                    ("humanoid15", (361, 64, 28), dict(grace_steps=2, write_back=True))])
def test_looped_clips_wrap_and_carry_the_root_along(skeleton, dims, extras):
    """A library that mixes looped and plain clips, run for more than two periods of the looped ones: time wraps, the
    cycle count (a fourth piece of per-env state, compared exactly) goes up, the root displacement of every completed
    cycle reaches the observation and the error terms, the plain clips truncate as before.  The simulator stand-in
    follows the continuous motion, so looped envs keep tracking well past the wrap."""
    sc = _scene("edge_loop_" + skeleton, dims, "f32", skeleton=skeleton, n_clips=4, frames=(61, 61), seed=9)
    flags = np.array([1, 0, 1, 1], np.uint8)
    sc.o_clips.set_cyclic(flags)
    sc.g_clips.set_cyclic(flags)
    n = 120
    p = Pair(sc, n, h_min=0.3, with_policy=False, **extras)
    p.reset_all()
    dur = np.float32(2.0)
    hist = []

    def consume(s, sim):
        if p.prev_o is not None:
            p.prev_o[:] = np.random.default_rng(1000 + s).standard_normal(p.prev_o.shape).astype(np.float32)
            p.prev_g.copy_(torch.from_numpy(p.prev_o))
        hist.append(p.env_step(s, sim))

    # the continuous time of an env = time inside the clip + completed cycles x duration
    W.rollout_inputs(sc.wl, sc.skel, sc.lib,
                     lambda: (p.o_env.clip_id, p.o_env.t.astype(np.float64) + p.o_env.cycle * float(dur)), consume, steps=130)
    looped = flags[p.o_env.clip_id].astype(bool)
    assert p.o_env.cycle[looped].max() >= 2 and np.all(p.o_env.cycle[~looped] == 0)
    assert any(((h["flags"] & 2) != 0).any() for h in hist)                  # plain clips truncated
    early = [h["reward"].mean() for h in hist[:10]]
    late = [h["reward"][looped].mean() for h in hist[-20:]]
    assert np.mean(late) > 0.5 * np.mean(early)                              # tracking as well after two wraps as before any
    sc.g_clips.set_cyclic(None)
    sc.o_clips.set_cyclic(None)
