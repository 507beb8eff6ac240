"""Pins for the oracle's extended observation (Section 6: "future reference end-effector frames, and
the previous action"), appended after the 24J+1 entries.  The expected values are closed forms of a
motion whose reference pose is known analytically (a root that translates and turns about z at
constant rates carrying rigid children), written out here with numpy; nothing calls the oracle to
produce them.
"""
import math

import numpy as np
import pytest

from oracle import oracle as O
from paper_2609_09821_b200 import workloads as W

FPS = 30.0
DT = np.float32(1.0 / 30.0)
V = np.array([0.7, -0.4, 0.0])          # root velocity, m/s
P0 = np.array([0.2, 0.1, 0.9])
OMEGA = 0.9                             # yaw rate, rad/s
OFFSETS = np.array([[0.0, 0.0, 0.0], [0.5, 0.1, 0.0], [-0.3, 0.2, 0.1]], np.float32)   # root and two children
REWARD = dict(W.REWARD_MULT, h_min=-np.inf, r_min=-np.inf)


def _rz(a):
    c, s = math.cos(a), math.sin(a)
    return np.array([[c, -s, 0.0], [s, c, 0.0], [0.0, 0.0, 1.0]])


def _scene(K=61, ee_ids=None):
    """Root + two children; the root moves at constant velocity and yaw rate, the children do not articulate."""
    parents = np.array([-1, 0, 0], np.int32)
    k = np.arange(K)
    root = (P0[None, :] + V[None, :] * (k[:, None] / FPS)).astype(np.float32)
    quat = np.zeros((K, 3, 4), np.float32)
    quat[:, :, 0] = 1.0
    quat[:, 0, 0] = np.cos(0.5 * OMEGA * k / FPS)
    quat[:, 0, 3] = np.sin(0.5 * OMEGA * k / FPS)
    skel = O.Skeleton(parents, OFFSETS, None, ee_ids)
    clips = O.Clips(skel, np.array([K], np.int32), np.array([FPS], np.float32), root, quat)
    return skel, clips


def _sim(n, yaw, root_xy, z=0.9):
    """SoA body state [13 J, n] with the root at (root_xy, z) turned by yaw; the children anywhere valid."""
    J = 3
    sim = np.zeros((13 * J, n), np.float32)
    for i in range(n):
        for j in range(J):
            sim[3 * j:3 * j + 3, i] = [root_xy[i][0] + 0.1 * j, root_xy[i][1], z[i] if np.ndim(z) else z]
            sim[3 * J + 4 * j:3 * J + 4 * j + 4, i] = [math.cos(yaw[i] / 2), 0.0, 0.0, math.sin(yaw[i] / 2)]
    return sim


def _expected_future(tau, yaw, origin_xy, body):
    """Nine entries of `body` at reference time tau seen from the heading frame (origin_xy, yaw)."""
    p_root = P0 + V * tau
    p = p_root + _rz(OMEGA * tau) @ OFFSETS[body].astype(np.float64)
    pos = _rz(-yaw) @ (p - np.array([origin_xy[0], origin_xy[1], 0.0]))
    a = OMEGA * tau - yaw
    return np.concatenate([pos, [math.cos(a), math.sin(a), 0.0], [0.0, 0.0, 1.0]])


def _env(skel, clips, n, t0, n_future, prev_action=None):
    cfg = O.make_env_config(float(DT), 3, REWARD, 0.3)
    env = O.Env(skel, clips, cfg, n)
    env.clip_id[:] = 0
    env.t[:] = t0
    env.ep_len[:] = 5
    D = env.set_obs_extension(n_future, prev_action)
    return env, D


def test_future_frames_follow_the_closed_form_in_frame_and_body_order():
    skel, clips = _scene()
    n, F = 3, 4
    t0 = np.array([0.2, 0.55, 1.0], np.float32)
    yaw, xy = [0.3, -1.1, 2.0], [(0.1, 0.2), (-0.4, 0.3), (1.0, -2.0)]
    env, D = _env(skel, clips, n, t0, F)
    assert D == 24 * 3 + 1 + (F - 1) * 9 * 2
    out = env.step(1, _sim(n, yaw, xy))
    assert not out["flags"].any()
    for i in range(n):
        t = np.float32(t0[i] + DT)                               # the env's time after the step
        assert env.t[i] == t
        base = 24 * 3 + 1
        for f in range(2, F + 1):
            tau = float(np.float32(t + np.float32(np.float32(f) * DT)))
            for slot, body in enumerate((1, 2)):                  # end effectors in body order
                got = out["obs"][i, base + ((f - 2) * 2 + slot) * 9: base + ((f - 2) * 2 + slot + 1) * 9]
                np.testing.assert_allclose(got, _expected_future(tau, yaw[i], xy[i], body), atol=2e-6)
        # frame 1 of the standard layout obeys the same formula (the extension continues it)
        tau1 = float(np.float32(t + DT))
        for body in (1, 2):
            got = out["obs"][i, 15 * 3 + 1 + 9 * body: 15 * 3 + 1 + 9 * body + 9]
            np.testing.assert_allclose(got, _expected_future(tau1, yaw[i], xy[i], body), atol=2e-6)


def test_end_effectors_keep_body_order_whatever_order_they_were_named_in():
    a = _scene(ee_ids=np.array([2, 1], np.int32))
    b = _scene(ee_ids=np.array([1, 2], np.int32))
    outs = []
    for skel, clips in (a, b):
        env, _ = _env(skel, clips, 1, np.array([0.4], np.float32), 3)
        outs.append(env.step(2, _sim(1, [0.5], [(0.0, 0.0)]))["obs"])
    np.testing.assert_array_equal(outs[0], outs[1])
    # a single named end effector: one block per frame, for that body
    skel, clips = _scene(ee_ids=np.array([2], np.int32))
    env, D = _env(skel, clips, 1, np.array([0.4], np.float32), 3)
    assert D == 24 * 3 + 1 + 2 * 9
    obs = env.step(2, _sim(1, [0.5], [(0.0, 0.0)]))["obs"][0]
    t = np.float32(np.float32(0.4) + DT)
    for f in (2, 3):
        tau = float(np.float32(t + np.float32(np.float32(f) * DT)))
        np.testing.assert_allclose(obs[73 + (f - 2) * 9: 73 + (f - 1) * 9], _expected_future(tau, 0.5, (0.0, 0.0), 2), atol=2e-6)


def test_future_frames_stop_at_the_end_of_the_clip():
    skel, clips = _scene(K=31)                                    # one second long
    dur = float(clips.duration(0))
    t0 = np.float32(dur - 2.5 * float(DT))                        # after the step 1.5 dt remain: frames 2.. are past the end
    env, _ = _env(skel, clips, 1, np.array([t0], np.float32), 4)
    out = env.step(1, _sim(1, [0.0], [(0.0, 0.0)]))
    assert out["flags"][0] == 0
    for f in (2, 3, 4):
        got = out["obs"][0, 73 + (f - 2) * 18: 73 + (f - 2) * 18 + 9]
        np.testing.assert_allclose(got, _expected_future(dur, 0.0, (0.0, 0.0), 1), atol=2e-6)


def test_previous_action_is_copied_and_cleared_on_reset():
    skel, clips = _scene()
    n, A = 4, 5
    prev = np.arange(n * A, dtype=np.float32).reshape(n, A) + 0.5
    cfg_reward = dict(REWARD, h_min=0.5)                          # envs whose root is below 0.5 m terminate
    cfg = O.make_env_config(float(DT), 3, cfg_reward, 0.3)
    env = O.Env(skel, clips, cfg, n)
    D = env.set_obs_extension(2, prev)
    assert D == 73 + 18 + A
    first = env.reset_all(0)
    assert not first[:, 73 + 18:].any()                           # nothing was done before the first observation
    env.clip_id[:] = 0
    env.t[:] = 0.3
    z = np.array([0.9, 0.2, 0.9, 0.1])
    out = env.step(1, _sim(n, [0.0] * n, [(0.0, 0.0)] * n, z))
    assert list(out["flags"] & 1) == [0, 1, 0, 1]
    tail = out["obs"][:, 73 + 18:]
    np.testing.assert_array_equal(tail[0], prev[0])
    np.testing.assert_array_equal(tail[2], prev[2])
    assert not tail[1].any() and not tail[3].any()
    assert out["obs"].shape[1] == D
    # the array is read at every step: what the caller writes into it shows up in the next observation
    prev[:] = -prev
    out = env.step(2, _sim(n, [0.0] * n, [(0.0, 0.0)] * n, 0.9))
    assert not out["flags"].any()
    np.testing.assert_array_equal(out["obs"][:, 73 + 18:], prev)


def test_extension_off_is_the_standard_row():
    skel, clips = _scene()
    env, D = _env(skel, clips, 2, np.array([0.2, 0.4], np.float32), 1)
    assert D == 73
    ext, _ = _env(skel, clips, 2, np.array([0.2, 0.4], np.float32), 3, np.ones((2, 4), np.float32))
    sim = _sim(2, [0.1, 0.2], [(0.0, 0.1), (0.3, 0.0)])
    a, b = env.step(1, sim.copy()), ext.step(1, sim.copy())
    np.testing.assert_array_equal(a["obs"], b["obs"][:, :73])
    np.testing.assert_array_equal(a["reward"], b["reward"])
