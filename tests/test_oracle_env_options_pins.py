"""Pins for the oracle's optional env semantics: early-termination grace steps and motion
randomisation of the reset state (both named in the paper's hyper-parameter table, both off by
default).  None of the checks restates the oracle's code path: they use the counter layout with an
independently written Box-Muller, rigid-body invariants, moments of the normal distribution, and
episode-length bookkeeping.
"""
import math

import numpy as np

from oracle import oracle as O
from paper_2609_09821_b200 import workloads as W


def _scene(kind="humanoid15", n_clips=3, frames=(40, 60)):
    skel = W.make_skeleton(kind, 0)
    lib = W.make_clip_library(skel["J"], n_clips, frames, 30.0, 0)
    o_skel = O.Skeleton(skel["parents"], skel["offsets"], skel["masses"])
    o_clips = O.Clips(o_skel, lib["n_frames"], lib["fps"], lib["root_pos"], lib["local_quat"])
    return skel, lib, o_skel, o_clips


def _qmul(a, b):
    w1, x1, y1, z1 = a
    w2, x2, y2, z2 = b
    return np.array([w1 * w2 - x1 * x2 - y1 * y2 - z1 * z2, w1 * x2 + x1 * w2 + y1 * z2 - z1 * y2,
                     w1 * y2 - x1 * z2 + y1 * w2 + z1 * x2, w1 * z2 + x1 * y2 - y1 * x2 + z1 * w2])


def _normals(seed, env, step, block):
    """First three Box-Muller normals of Philox block (env, step, 2, block), written out here."""
    x = O.philox([env, step, 2, block], [seed & 0xFFFFFFFF, seed >> 32])
    u1 = (float(x[0] >> 8) + 1.0) * 2.0 ** -24
    u2 = float(x[1] >> 8) * 2.0 ** -24
    u3 = (float(x[2] >> 8) + 1.0) * 2.0 ** -24
    u4 = float(x[3] >> 8) * 2.0 ** -24
    r1, r2 = math.sqrt(-2 * math.log(u1)), math.sqrt(-2 * math.log(u3))
    return np.array([r1 * math.cos(2 * math.pi * u2), r1 * math.sin(2 * math.pi * u2), r2 * math.cos(2 * math.pi * u4)])


def test_zero_std_leaves_the_reference_state():
    skel, lib, o_skel, o_clips = _scene()
    cfg = O.make_env_config(1 / 30, 5, W.REWARD_MULT, 0.3)
    ref = O.reference_state(o_skel, o_clips, 1, 0.4)
    got = O.reset_state(o_skel, o_clips, cfg, 7, 3, 1, 0.4)
    for k in ("p", "q", "v", "w"):
        np.testing.assert_array_equal(got[k], ref[k])


def test_noise_uses_the_stated_counters_and_rotates_in_the_joint_frame():
    skel, lib, o_skel, o_clips = _scene()
    std, seed, env, step = 0.05, 0x1234ABCD5678, 11, 4
    cfg = O.make_env_config(1 / 30, seed, W.REWARD_MULT, 0.3, reset_noise_std=std)
    ref = O.reference_state(o_skel, o_clips, 2, 0.7)
    got = O.reset_state(o_skel, o_clips, cfg, env, step, 2, 0.7)
    J = skel["J"]
    for j in range(J):
        n = std * _normals(seed, env, step, j)
        th = np.linalg.norm(n)
        dq = np.concatenate([[math.cos(th / 2)], math.sin(th / 2) * n / th])
        np.testing.assert_allclose(got["ql"][j], _qmul(ref["ql"][j], dq), atol=1e-12)
    np.testing.assert_allclose(got["p"][0], ref["p"][0] + std * _normals(seed, env, step, J), atol=1e-12)
    # another env or step draws other numbers
    other = O.reset_state(o_skel, o_clips, cfg, env + 1, step, 2, 0.7)
    assert np.abs(other["ql"] - got["ql"]).max() > 1e-4
    other = O.reset_state(o_skel, o_clips, cfg, env, step + 1, 2, 0.7)
    assert np.abs(other["ql"] - got["ql"]).max() > 1e-4


def test_randomised_state_is_a_rigid_pose_of_the_same_skeleton():
    """Bone lengths are kept, world rotations are the products of the local ones, and the velocity of
    a child origin is the parent's plus omega x arm."""
    skel, lib, o_skel, o_clips = _scene("smpl24")
    cfg = O.make_env_config(1 / 30, 9, W.REWARD_MULT, 0.3, reset_noise_std=0.2)
    st = O.reset_state(o_skel, o_clips, cfg, 3, 8, 0, 0.31)
    par = skel["parents"]
    for j in range(1, skel["J"]):
        a = par[j]
        arm = st["p"][j] - st["p"][a]
        np.testing.assert_allclose(np.linalg.norm(arm), np.linalg.norm(skel["offsets"][j]), atol=1e-6)
        np.testing.assert_allclose(st["q"][j], _qmul(st["q"][a], st["ql"][j]), atol=1e-12)
        np.testing.assert_allclose(st["v"][j], st["v"][a] + np.cross(st["w"][a], arm), atol=1e-10)
    np.testing.assert_allclose(np.linalg.norm(st["q"], axis=1), 1.0, atol=1e-12)


def test_noise_moments():
    """Over many envs: joint rotation angles have E|n|^2 = 3 std^2, the root shift has mean 0 and
    variance std^2 per axis, and two joints are uncorrelated."""
    skel, lib, o_skel, o_clips = _scene()
    std = 0.02                                            # the paper's baseline value
    cfg = O.make_env_config(1 / 30, 1, W.REWARD_MULT, 0.3, reset_noise_std=std)
    ref = O.reference_state(o_skel, o_clips, 0, 0.5)
    ang2, shift, n3, n5 = [], [], [], []
    for env in range(3000):
        st = O.reset_state(o_skel, o_clips, cfg, env, 1, 0, 0.5)
        rel = np.array([_qmul(ref["ql"][j] * [1, -1, -1, -1], st["ql"][j]) for j in range(skel["J"])])
        rv = 2 * rel[:, 1:] / np.maximum(rel[:, :1], 1e-9)            # small angles: n ~ 2 vec / w
        ang2.append((rv ** 2).sum(axis=1))
        n3.append(rv[3, 0]); n5.append(rv[5, 0])
        shift.append(st["p"][0] - ref["p"][0])
    ang2, shift = np.array(ang2), np.array(shift)
    np.testing.assert_allclose(ang2.mean(), 3 * std ** 2, rtol=0.03)
    np.testing.assert_allclose(shift.std(axis=0), std, rtol=0.05)
    assert np.abs(shift.mean(axis=0)).max() < 4 * std / math.sqrt(3000)
    assert abs(np.corrcoef(n3, n5)[0, 1]) < 0.08


def test_reset_env_observes_and_writes_back_the_randomised_state():
    skel, lib, o_skel, o_clips = _scene()
    wl = W.WORKLOADS["cfg1_tiny64"]
    n, J = 32, skel["J"]
    cfg = O.make_env_config(wl.dt, 3, W.REWARD_MULT, 10.0, write_back_reset=True, reset_noise_std=0.05)   # h_min 10: all reset
    env = O.Env(o_skel, o_clips, cfg, n)
    env.reset_all(0)
    sim = W.synth_sim_state(skel, lib, env.clip_id, env.t.astype(np.float64) + wl.dt, 1, wl)
    out = env.step(1, sim)
    assert (out["flags"] & 1).all()
    for e in (0, 17, 31):
        st = O.reset_state(o_skel, o_clips, cfg, e, 1, int(env.clip_id[e]), float(env.t[e]))
        pos, quat, lin, ang = W.split_sim(sim, J)
        np.testing.assert_allclose(pos[:, e].reshape(J, 3), st["p"], atol=1e-6)
        np.testing.assert_allclose(quat[:, e].reshape(J, 4), st["q"], atol=1e-6)
        np.testing.assert_allclose(lin[:, e].reshape(J, 3), st["v"], atol=1e-5)
        np.testing.assert_allclose(ang[:, e].reshape(J, 3), st["w"], atol=1e-5)
        # the root's observed position is (0, 0, z) in its own heading frame, z of the shifted root
        np.testing.assert_allclose(out["obs"][e, :3], [0.0, 0.0, st["p"][0][2]], atol=1e-12)


def test_grace_steps_delay_early_termination_but_not_truncation():
    skel, lib, o_skel, o_clips = _scene(n_clips=2, frames=(12, 12))          # 11 intervals: truncation comes early
    wl = W.WORKLOADS["cfg1_tiny64"]
    n, G = 16, 3
    cfg = O.make_env_config(wl.dt, 2, W.REWARD_MULT, 10.0, grace_steps=G)     # h_min 10: every step would terminate
    env = O.Env(o_skel, o_clips, cfg, n)
    env.reset_all(0)
    lens = [env.ep_len.copy()]
    for s in range(1, 14):
        before = env.ep_len.copy()
        sim = W.synth_sim_state(skel, lib, env.clip_id, env.t.astype(np.float64) + wl.dt, s, wl)
        out = env.step(s, sim)
        term, trunc = out["flags"] & 1, out["flags"] >> 1
        np.testing.assert_array_equal(term, (before >= G).astype(np.uint8))
        # truncation is decided by the clock alone
        assert ((trunc == 1) | (term == 1) == (env.ep_len == 0)).all()
        lens.append(env.ep_len.copy())
    lens = np.array(lens)
    assert lens.max() == G                               # an episode never survives G + 1 steps here
    assert (np.diff(lens, axis=0)[lens[1:] > 0] == 1).all()
    # G = 0 is the old behaviour: everything terminates at once
    env0 = O.Env(o_skel, o_clips, O.make_env_config(wl.dt, 2, W.REWARD_MULT, 10.0), n)
    env0.reset_all(0)
    sim = W.synth_sim_state(skel, lib, env0.clip_id, env0.t.astype(np.float64) + wl.dt, 1, wl)
    assert (env0.step(1, sim)["flags"] & 1).all()


# ---------------------------------------------------------------- adaptive episode initialisation
def test_cumulative_table_closed_forms():
    np.testing.assert_array_equal(O.reset_cdf([1, 1, 2]), [2 ** 30, 2 ** 31, 2 ** 32])
    np.testing.assert_array_equal(O.reset_cdf([0, 3, 0, 1, 0]), [0, 3 * 2 ** 30, 3 * 2 ** 30, 2 ** 32, 2 ** 32])
    np.testing.assert_array_equal(O.reset_cdf([5.0]), [2 ** 32])
    T = O.reset_cdf(np.ones(7))
    np.testing.assert_array_equal(T[:-1], [(k * 2 ** 32) // 7 for k in range(1, 7)])
    for bad in ([0, 0], [1, -1], [np.nan, 1], [np.inf, 1]):
        try:
            O.reset_cdf(bad)
        except ValueError:
            continue
        raise AssertionError("accepted %r" % (bad,))


def _binned_env(weights, n=4000, seed=11, frames=(40, 60), h_min=0.3):
    skel, lib, o_skel, o_clips = _scene(n_clips=3, frames=frames)
    cfg = O.make_env_config(1 / 30, seed, W.REWARD_MULT, h_min)
    env = O.Env(o_skel, o_clips, cfg, n)
    env.set_reset_bins(np.asarray(weights).shape[1], weights)
    return skel, lib, o_clips, env


def test_binned_draws_follow_the_weights_and_stay_inside_their_bin():
    import scipy.stats
    w = np.array([[1, 0, 2, 1], [0, 0, 0, 4], [3, 1, 0, 0]], np.float32)
    skel, lib, o_clips, env = _binned_env(w, n=20000)
    env.reset_all(0)
    B = w.shape[1]
    span = np.array([o_clips.duration(c) for c in range(3)], np.float64) - 1 / 30
    b = np.minimum(np.floor(env.t / (span[env.clip_id] / B) * (1 + 1e-9)).astype(int), B - 1)
    counts = np.zeros_like(w)
    np.add.at(counts, (env.clip_id, b), 1)
    assert (counts[w == 0] == 0).all()                                   # weight 0 is never drawn
    expect = w / w.sum() * env.n
    chi2 = ((counts - expect)[w > 0] ** 2 / expect[w > 0]).sum()
    assert chi2 < scipy.stats.chi2.ppf(0.999, (w > 0).sum() - 1)
    # uniform inside a bin: position within the bin against U(0, 1)
    sel = (env.clip_id == 1)
    frac = env.t[sel] / (span[1] / B) - 3
    assert frac.min() >= -1e-6 and frac.max() <= 1 + 1e-6
    assert scipy.stats.kstest(np.clip(frac, 0, 1), "uniform").pvalue > 1e-3
    assert (env.t <= span[env.clip_id] + 1e-9).all()
    np.testing.assert_array_equal(env.stat_starts.reshape(w.shape), counts.astype(np.uint32))


def test_one_equal_bin_per_clip_is_the_uniform_distribution_over_clips():
    import scipy.stats
    skel, lib, o_clips, env = _binned_env(np.ones((3, 1), np.float32), n=30000)
    env.reset_all(0)
    counts = np.bincount(env.clip_id, minlength=3)
    assert scipy.stats.chisquare(counts).pvalue > 1e-3
    span = np.array([o_clips.duration(c) for c in range(3)], np.float64) - 1 / 30
    assert scipy.stats.kstest(env.t / span[env.clip_id], "uniform").pvalue > 1e-3


def test_failure_and_start_counts_add_up():
    wl = W.WORKLOADS["cfg1_tiny64"]
    B = 5
    skel, lib, o_clips, env = _binned_env(np.ones((3, B), np.float32), n=600, h_min=W.ROOT_HEIGHT)
    env.reset_all(0)
    n_term = n_reset = 0
    fail_bins = np.zeros((3, B), np.int64)
    span = np.array([o_clips.duration(c) for c in range(3)], np.float64) - wl.dt
    for s in range(1, 9):
        clip_before = env.clip_id.copy()
        t1 = (env.t + np.float32(wl.dt)).astype(np.float64)
        sim = W.synth_sim_state(skel, lib, env.clip_id, env.t.astype(np.float64) + wl.dt, s, wl)
        out = env.step(s, sim, want_terms=False)
        term = (out["flags"] & 1) == 1
        n_term += int(term.sum())
        n_reset += int((out["flags"] != 0).sum())
        pos = t1 / (span[clip_before] / B)
        safe = term & (np.abs(pos - np.round(pos)) > 1e-4)               # away from bin edges the bin is unambiguous
        np.add.at(fail_bins, (clip_before[safe], np.minimum(np.floor(pos[safe]).astype(int), B - 1)), 1)
        assert safe.sum() >= term.sum() - 2
    assert n_term > 100
    assert int(env.stat_failures.sum()) == n_term
    assert int(env.stat_starts.sum()) == env.n + n_reset
    assert np.abs(env.stat_failures.reshape(3, B).astype(np.int64) - fail_bins).sum() <= 16


def test_adaptation_draws_bins_in_proportion_to_failures_plus_floor():
    """After adapt_reset_bins the probability of a (clip, bin) is (failures + floor) / sum, to within the
    2^-32 granularity of the table; a large floor tends to the uniform table; the counts restart."""
    import scipy.stats
    B = 4
    skel, lib, o_clips, env = _binned_env(np.ones((3, B), np.float32), n=30000)
    fails = np.array([[0, 5, 0, 1], [40, 0, 0, 0], [2, 2, 2, 100]], np.uint32)
    env.stat_failures[:] = fails.ravel()
    env.stat_starts[:] = 7
    floor = 0.5
    w = env.adapt_reset_bins(floor)
    assert not env.stat_failures.any() and not env.stat_starts.any()
    want = (fails.ravel().astype(np.float64) + floor)
    np.testing.assert_array_equal(w, want.astype(np.float32))
    T = env.reset_cdf.astype(np.float64)
    prob = np.diff(np.concatenate([[0.0], T])) / 2.0 ** 32
    np.testing.assert_allclose(prob, want / want.sum(), atol=2.0 ** -31)
    # the draws follow it
    env.reset_all(3)
    counts = env.stat_starts.astype(np.float64)
    expect = want / want.sum() * env.n
    assert ((counts - expect) ** 2 / expect).sum() < scipy.stats.chi2.ppf(0.999, want.size - 1)
    # keeping the counts, and a floor that swamps them
    env.stat_failures[:] = fails.ravel()
    env.adapt_reset_bins(1e9, clear=False)
    np.testing.assert_array_equal(env.stat_failures, fails.ravel())
    prob = np.diff(np.concatenate([[0.0], env.reset_cdf.astype(np.float64)])) / 2.0 ** 32
    np.testing.assert_allclose(prob, 1.0 / want.size, rtol=1e-6)
