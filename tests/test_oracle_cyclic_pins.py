"""Pins for the oracle's cyclic clips (periodic motions played in a loop: the time wraps at the clip's end, the
root translation of each completed cycle accumulates, the clip never truncates).

The seeded clips are exactly periodic when they span one period of their slowest harmonic (61 keyframes at
30 Hz = 2 s): the last keyframe is the first one moved by (2, 0, 0).  A "simulator" that tracks the looped
reference perfectly (state built here from the non-cyclic reference plus n times the cycle displacement read off
the keyframes, not from the oracle's own cyclic code) must then score reward 1 at every step, wraps included;
what the observation says about the next frames must stay continuous through the wrap; the observation repeats
after one period; time stays inside the clip and the cycle counter counts."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2609_09821_b200 import workloads as W

DT = 1.0 / 30.0


def _scene(flags=(1, 0, 1), n_future=1):
    skel = W.make_skeleton("humanoid15", 3)
    lib = W.make_clip_library(15, 3, (61, 61), 30.0, seed=4)
    osk = O.Skeleton(skel["parents"], skel["offsets"], skel["masses"])
    ocl = O.Clips(osk, lib["n_frames"], lib["fps"], lib["root_pos"], lib["local_quat"])
    ocl.set_cyclic(np.asarray(flags, np.uint8))
    shift = np.array([lib["root_pos"][lib["frame_start"][c] + 60] - lib["root_pos"][lib["frame_start"][c]] for c in range(3)],
                     np.float64)
    return skel, lib, osk, ocl, shift


def _tracking_state(osk, ocl, shift, clip, t, cyc):
    """Body state [13 J] that equals the looped reference: the plain reference at (clip, t) moved by cyc cycles."""
    r = O.reference_state(osk, ocl, int(clip), np.float32(t))
    p = r["p"] + cyc * shift[clip]
    return np.concatenate([p.ravel(), r["q"].ravel(), r["v"].ravel(), r["w"].ravel()])


def _advance(t, cyc, dur, cyclic):
    t1 = np.float32(np.float32(t) + np.float32(DT))
    if cyclic and t1 >= dur:
        return np.float32(t1 - dur), cyc + 1
    return t1, cyc


def test_the_seeded_61_frame_clips_are_one_exact_period():
    skel, lib, osk, ocl, shift = _scene()
    for c in range(3):
        s = lib["frame_start"][c]
        np.testing.assert_allclose(shift[c], [2.0, 0.0, 0.0], atol=1e-6)
        np.testing.assert_allclose(np.abs((lib["local_quat"][s] * lib["local_quat"][s + 60]).sum(-1)), 1.0, atol=1e-6)


def test_perfect_tracking_of_a_looped_clip_scores_one_through_every_wrap():
    skel, lib, osk, ocl, shift = _scene()
    n = 48
    env = O.Env(osk, ocl, O.make_env_config(DT, 11, W.REWARD_MULT, -10.0), n)
    obs = env.reset_all(0)
    dur = np.float32(2.0)
    first_obs = {}
    wraps = np.zeros(n, int)
    for s in range(1, 151):                       # two and a half cycles
        clip, t, cyc = env.clip_id.copy(), env.t.copy(), env.cycle.copy()
        sim = np.zeros((13 * 15, n), np.float32)
        want_t, want_cyc = t.copy(), cyc.copy()
        for i in range(n):
            want_t[i], want_cyc[i] = _advance(t[i], cyc[i], dur, bool(ocl.cyclic[clip[i]]))
            sim[:, i] = _tracking_state(osk, ocl, shift, clip[i], want_t[i], want_cyc[i])
        out = env.step(s, sim)
        cyclic = ocl.cyclic[clip].astype(bool)
        # reward 1 everywhere the state is the (looped) reference -- a wrap without the cycle displacement, or with a
        # wrong one, would put the whole character 2 m away from the reference
        np.testing.assert_allclose(out["reward"][cyclic], 1.0, atol=1e-6)
        assert np.all((out["flags"][cyclic] & 2) == 0)                      # a looped clip never truncates
        keep = out["flags"] == 0
        np.testing.assert_array_equal(env.t[keep].view(np.uint32), want_t[keep].view(np.uint32))
        np.testing.assert_array_equal(env.cycle[keep], want_cyc[keep])
        assert np.all(env.cycle[~keep] == 0) and np.all(env.cycle[~cyclic & keep] == 0)
        assert np.all(env.t[cyclic & keep] < dur)
        wraps += (want_cyc > cyc) & keep
        # the observation of a looped env repeats one period (60 steps) later
        for i in np.nonzero(cyclic & keep)[0]:
            if s in first_obs.get(i, {}):
                continue
            first_obs.setdefault(i, {})[s] = out["obs"][i]
            if s - 60 in first_obs[i]:
                np.testing.assert_allclose(out["obs"][i], first_obs[i][s - 60], atol=2e-4)
    looped = ocl.cyclic[env.clip_id].astype(bool) & (env.ep_len == 150)
    # 150 steps are two and a half periods: two or three wraps depending on the starting phase
    assert looped.sum() >= 10 and np.all(wraps[looped] == env.cycle[looped]) and set(wraps[looped]) == {2, 3}
    # the clip that is not looped truncated and reset its envs as before
    assert (env.ep_len < 150).any()


def test_look_ahead_targets_stay_continuous_through_the_wrap():
    """The observed target of the root one (and, with further frames, two) intervals ahead is the root's own velocity
    times the look-ahead, whether or not the look-ahead crosses the end of the clip."""
    skel, lib, osk, ocl, shift = _scene(flags=(1, 1, 1))
    n = 8
    env = O.Env(osk, ocl, O.make_env_config(DT, 5, W.REWARD_MULT, -10.0), n)
    ee = osk.ee_ids
    D = env.set_obs_extension(3, None)
    env.reset_all(0)
    dur = np.float32(2.0)
    crossed = 0
    for s in range(1, 130):
        clip, t, cyc = env.clip_id.copy(), env.t.copy(), env.cycle.copy()
        sim = np.zeros((13 * 15, n), np.float32)
        for i in range(n):
            t1, c1 = _advance(t[i], cyc[i], dur, True)
            sim[:, i] = _tracking_state(osk, ocl, shift, clip[i], t1, c1)
        out = env.step(s, sim)
        for i in range(n):
            o = out["obs"][i]
            vel = o[9:12]                                        # the root's heading-local velocity
            tgt = o[15 * 15 + 1:15 * 15 + 4] - o[0:3]            # root target one interval ahead, relative to the root
            assert np.abs(tgt - vel * DT).max() < 2e-3, (s, i, tgt, vel * DT)
            crossed += env.t[i] + DT >= dur
    assert crossed >= n                                          # the look-ahead did cross the end of the clip
    # further frames of the end effectors: the step from frame 2 to frame 3 is as small as any other
    blk = out["obs"][:, 24 * 15 + 1:24 * 15 + 1 + 2 * 9 * len(ee)].reshape(n, 2, len(ee), 9)
    assert np.abs(blk[:, 1, :, :3] - blk[:, 0, :, :3]).max() < 0.5


def test_flags_cleared_means_no_loop():
    skel, lib, osk, ocl, shift = _scene(flags=(0, 0, 0))
    env = O.Env(osk, ocl, O.make_env_config(DT, 1, W.REWARD_MULT, -10.0), 16)
    env.reset_all(0)
    trunc = 0
    for s in range(1, 70):
        sim = W.synth_sim_state(skel, lib, env.clip_id, env.t.astype(np.float64) + DT, s, W.WORKLOADS["cfg1_tiny64"])
        trunc += int((env.step(s, sim)["flags"] & 2).sum())
        assert np.all(env.cycle == 0)
    assert trunc >= 16
