"""Pins for the CPU oracle: each check compares it with something other than
itself -- published known answers, closed forms, 3x3-matrix brute force,
library routines (scipy expm/logm, torch linear), invariants and statistics.
"""
import math
import os

import numpy as np
import pytest
import scipy.linalg
import scipy.stats

from oracle import oracle as O
from paper_2609_09821_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ helpers
def rodrigues(axis, angle):
    """Rotation matrix from axis-angle, written with matrices only."""
    a = np.asarray(axis, float)
    a = a / np.linalg.norm(a)
    K = np.array([[0, -a[2], a[1]], [a[2], 0, -a[0]], [-a[1], a[0], 0]])
    return np.eye(3) + math.sin(angle) * K + (1 - math.cos(angle)) * K @ K


def axis_angle_quat(axis, angle):
    a = np.asarray(axis, float)
    a = a / np.linalg.norm(a)
    return np.concatenate([[math.cos(angle / 2)], math.sin(angle / 2) * a])


def quat_matrix(q):
    """Matrix of a unit quaternion via its action on the basis vectors (uses the oracle's rotate
    only to read columns); used where the matrix route is the independent part (composition)."""
    return np.stack([O.quat_rotate(q, e) for e in np.eye(3)], axis=1)


def random_unit_quats(rng, *shape):
    q = rng.standard_normal(shape + (4,))
    return q / np.linalg.norm(q, axis=-1, keepdims=True)


def tiny_scene(J=3, K=6, parents=None, seed=3, C=1, static=False, fps=30.0, spread=0.25):
    rng = np.random.default_rng(seed)
    parents = np.asarray(parents if parents is not None else [-1] + list(range(J - 1)), np.int32)
    J = len(parents)
    offsets = rng.uniform(-0.4, 0.4, size=(J, 3)).astype(np.float32)
    offsets[0] = 0
    masses = rng.uniform(1, 5, size=J).astype(np.float32)
    n_frames = np.full(C, K, np.int32)
    total = int(n_frames.sum())
    quat = random_unit_quats(rng, total, J)
    # keep consecutive keyframes close so that slerp is well conditioned
    base = random_unit_quats(rng, 1, J)
    quat = base + spread * quat
    quat /= np.linalg.norm(quat, axis=-1, keepdims=True)
    root = rng.uniform(-1, 1, size=(total, 3))
    root[:, 2] += 1.0
    if static:
        quat[:] = quat[0]
        root[:] = root[0]
    skel = O.Skeleton(parents, offsets, masses)
    clips = O.Clips(skel, n_frames, np.full(C, fps, np.float32), root.astype(np.float32),
                    quat.astype(np.float32))
    return dict(skel=skel, clips=clips, parents=parents, offsets=offsets, masses=masses,
                quat=quat.astype(np.float32), root=root.astype(np.float32), K=K, fps=fps)


def matrix_fk(parents, offsets, root_p, local_R):
    """Brute-force forward kinematics with 3x3 matrices."""
    J = len(parents)
    R = [None] * J
    p = [None] * J
    R[0], p[0] = local_R[0], np.asarray(root_p, float)
    for j in range(1, J):
        a = parents[j]
        R[j] = R[a] @ local_R[j]
        p[j] = p[a] + R[a] @ offsets[j].astype(float)
    return np.array(p), R


def scene_from_workload(name, n=None):
    wl = W.WORKLOADS[name]
    skel, lib, pol = W.build_scene(wl)
    osk = O.Skeleton(skel["parents"], skel["offsets"], skel["masses"])
    ocl = O.Clips(osk, lib["n_frames"], lib["fps"], lib["root_pos"], lib["local_quat"])
    return wl, skel, lib, pol, osk, ocl


# ------------------------------------------------------------------ Philox
def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) if l[0] != "#"]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        assert list(O.philox(v[0:4], v[4:6])) == v[6:10]


def test_philox_counter_words_are_distinct_streams():
    a = O.philox([5, 7, 0, 0], [1, 2])
    assert not np.array_equal(a, O.philox([7, 5, 0, 0], [1, 2]))
    assert not np.array_equal(a, O.philox([5, 7, 1, 0], [1, 2]))
    assert not np.array_equal(a, O.philox([5, 7, 0, 0], [2, 1]))


# ------------------------------------------------------------------ quaternions
def test_rotate_quarter_turn_about_z():
    q = axis_angle_quat([0, 0, 1], math.pi / 2)
    np.testing.assert_allclose(O.quat_rotate(q, [1, 0, 0]), [0, 1, 0], atol=1e-15)
    np.testing.assert_allclose(O.quat_rotate(q, [0, 1, 0]), [-1, 0, 0], atol=1e-15)


def test_rotate_matches_rodrigues_and_mul_is_composition():
    rng = np.random.default_rng(0)
    for _ in range(20):
        ax1, ax2 = rng.standard_normal(3), rng.standard_normal(3)
        a1, a2 = rng.uniform(-3, 3, 2)
        q1, q2 = axis_angle_quat(ax1, a1), axis_angle_quat(ax2, a2)
        v = rng.standard_normal(3)
        np.testing.assert_allclose(O.quat_rotate(q1, v), rodrigues(ax1, a1) @ v, atol=1e-13)
        np.testing.assert_allclose(O.quat_rotate(O.quat_mul(q1, q2), v),
                                   rodrigues(ax1, a1) @ rodrigues(ax2, a2) @ v, atol=1e-13)


def test_geodesic_angle_and_log():
    rng = np.random.default_rng(1)
    for phi in [0.0, 1e-9, 0.3, 1.0, 2.5, math.pi - 1e-6, math.pi]:
        ax = rng.standard_normal(3)
        ax /= np.linalg.norm(ax)
        q = axis_angle_quat(ax, phi)
        assert abs(O.geodesic_angle(q) - phi) < 1e-12
        assert abs(O.geodesic_angle(-q) - phi) < 1e-12
        np.testing.assert_allclose(2 * O.quat_log(q), phi * ax, atol=1e-12)
        np.testing.assert_allclose(2 * O.quat_log(-q), phi * ax, atol=1e-12)
    # past pi the shortest arc goes the other way round
    q = axis_angle_quat([0, 0, 1], math.pi + 0.4)
    np.testing.assert_allclose(2 * O.quat_log(q), [0, 0, -(math.pi - 0.4)], atol=1e-12)


# ------------------------------------------------------------------ slerp
def test_slerp_endpoints_norm_and_sign():
    rng = np.random.default_rng(2)
    for _ in range(50):
        q0, q1 = random_unit_quats(rng, 2)
        a = rng.uniform()
        s = O.slerp(q0, q1, a)
        assert abs(np.linalg.norm(s) - 1) < 1e-14
        np.testing.assert_allclose(O.slerp(q0, q1, 0.0), q0, atol=1e-14)
        e1 = O.slerp(q0, q1, 1.0)
        assert min(np.abs(e1 - q1).max(), np.abs(e1 + q1).max()) < 1e-14
        # negating either keyframe gives the same rotation
        for s2 in (O.slerp(-q0, q1, a), O.slerp(q0, -q1, a)):
            assert min(np.abs(s2 - s).max(), np.abs(s2 + s).max()) < 1e-13


def test_slerp_common_axis_blends_angle_linearly():
    ax = np.array([0.3, -0.5, 0.8])
    for a0, a1, al in [(0.2, 1.4, 0.25), (-1.0, 0.5, 0.7), (0.1, 0.1 + 1e-8, 0.5), (3.0, 3.0 - 2.9, 0.9)]:
        s = O.slerp(axis_angle_quat(ax, a0), axis_angle_quat(ax, a1), al)
        want = rodrigues(ax, (1 - al) * a0 + al * a1)
        np.testing.assert_allclose(quat_matrix(s), want, atol=1e-9)


def test_slerp_matches_matrix_exponential():
    rng = np.random.default_rng(4)
    for _ in range(10):
        ax0, ax1 = rng.standard_normal(3), rng.standard_normal(3)
        a0, a1 = rng.uniform(-1.2, 1.2, 2)
        R0, R1 = rodrigues(ax0, a0), rodrigues(ax1, a1)
        al = rng.uniform()
        want = R0 @ scipy.linalg.expm(al * np.real(scipy.linalg.logm(R0.T @ R1)))
        got = quat_matrix(O.slerp(axis_angle_quat(ax0, a0), axis_angle_quat(ax1, a1), al))
        np.testing.assert_allclose(got, want, atol=1e-9)


# ------------------------------------------------------------------ lookup
def test_lookup_index_on_keyframes_and_at_the_end():
    K = 60
    for k in range(K - 1):
        kk, a = O.lookup_index(np.float32(k) / np.float32(30), 30.0, K)
        f = np.float32(np.float32(k) / np.float32(30)) * np.float32(30)
        assert kk == min(int(math.floor(f)), K - 2)
        assert abs(kk + a - k) < 4e-6
    kk, a = O.lookup_index((K - 1) / 30.0, 30.0, K)
    assert kk == K - 2 and abs(a - 1) < 4e-6
    kk, a = O.lookup_index(100.0, 30.0, K)          # beyond the end: clamps to the last pose
    assert kk == K - 2 and a == 1.0
    kk, a = O.lookup_index(0.515625, 30.0, K)       # 15.46875 exactly
    assert kk == 15 and a == 0.46875


def test_reference_reproduces_keyframes():
    sc = tiny_scene(J=4, K=7)
    for k in range(sc["K"]):
        t = np.float32(k) / np.float32(sc["fps"])
        r = O.reference_state(sc["skel"], sc["clips"], 0, t)
        qk = sc["quat"][k].astype(float)
        qk /= np.linalg.norm(qk, axis=-1, keepdims=True)
        for j in range(4):
            assert min(np.abs(r["ql"][j] - qk[j]).max(), np.abs(r["ql"][j] + qk[j]).max()) < 2e-6
        np.testing.assert_allclose(r["p"][0], sc["root"][k], atol=5e-6)


# ------------------------------------------------------------------ FK
def test_fk_straight_chain_sums_offsets():
    J = 5
    parents = np.array([-1, 0, 1, 2, 3], np.int32)
    offsets = np.array([[0, 0, 0], [0.1, 0, 0], [0.2, 0.05, 0], [0, 0.3, 0.1], [0.05, 0.05, 0.05]], np.float32)
    skel = O.Skeleton(parents, offsets)
    quat = np.zeros((3, J, 4), np.float32)
    quat[..., 0] = 1
    root = np.array([[1, 2, 3]] * 3, np.float32)
    clips = O.Clips(skel, [3], [30.0], root, quat)
    r = O.reference_state(skel, clips, 0, 0.02)
    np.testing.assert_allclose(r["p"], root[0] + np.cumsum(offsets.astype(float), axis=0), atol=1e-15)
    np.testing.assert_allclose(r["q"], np.tile([1.0, 0, 0, 0], (J, 1)), atol=1e-15)
    np.testing.assert_allclose(r["v"], 0, atol=1e-15)
    np.testing.assert_allclose(r["com"], r["p"].mean(axis=0), atol=1e-15)   # unit masses


def test_fk_one_joint_quarter_turn():
    parents = np.array([-1, 0, 1], np.int32)
    offsets = np.array([[0, 0, 0], [1, 0, 0], [1, 0, 0]], np.float32)
    skel = O.Skeleton(parents, offsets)
    quat = np.zeros((2, 3, 4), np.float32)
    quat[..., 0] = 1
    quat[:, 1] = axis_angle_quat([0, 0, 1], math.pi / 2).astype(np.float32)
    clips = O.Clips(skel, [2], [30.0], np.zeros((2, 3), np.float32), quat)
    r = O.reference_state(skel, clips, 0, 0.0)
    # body 1 sits at the root's +x; its own quarter turn swings its child to +y
    np.testing.assert_allclose(r["p"], [[0, 0, 0], [1, 0, 0], [1, 1, 0]], atol=1e-7)


@pytest.mark.parametrize("parents", [[-1], [-1, 0], [-1, 0, 0], [-1, 0, 1, 1, 0, 4], W.PARENTS_15, W.PARENTS_24])
def test_fk_against_matrix_brute_force(parents):
    sc = tiny_scene(parents=parents, K=5, seed=len(parents))
    J = len(parents)
    for t in [0.0, 0.0171, 0.05, 4 / 30.0]:
        k, al = O.lookup_index(t, 30.0, sc["K"])
        q0 = sc["quat"][k].astype(float)
        q1 = sc["quat"][k + 1].astype(float)
        q0 /= np.linalg.norm(q0, axis=-1, keepdims=True)
        q1 /= np.linalg.norm(q1, axis=-1, keepdims=True)
        local_R = []
        for j in range(J):
            R0, R1 = quat_matrix(q0[j]), quat_matrix(q1[j])
            local_R.append(R0 @ scipy.linalg.expm(al * np.real(scipy.linalg.logm(R0.T @ R1))))
        root = (1 - al) * sc["root"][k].astype(float) + al * sc["root"][k + 1].astype(float)
        p, R = matrix_fk(sc["parents"], sc["offsets"], root, local_R)
        r = O.reference_state(sc["skel"], sc["clips"], 0, t)
        np.testing.assert_allclose(r["p"], p, atol=1e-8)
        for j in range(J):
            np.testing.assert_allclose(quat_matrix(r["q"][j]), R[j], atol=1e-8)
        m = sc["masses"].astype(float)
        np.testing.assert_allclose(r["com"], (m[:, None] * p).sum(0) / m.sum(), atol=1e-9)


@pytest.mark.parametrize("parents", [[-1, 0, 1], W.PARENTS_15, W.PARENTS_24])
def test_velocities_match_central_differences(parents):
    sc = tiny_scene(parents=parents, K=30, seed=11, spread=0.04)
    t, d = 0.515625, 2.0 ** -12          # both exactly representable, inside one keyframe interval
    r = O.reference_state(sc["skel"], sc["clips"], 0, t)
    ra = O.reference_state(sc["skel"], sc["clips"], 0, t - d)
    rb = O.reference_state(sc["skel"], sc["clips"], 0, t + d)
    v_fd = (rb["p"] - ra["p"]) / (2 * d)
    np.testing.assert_allclose(r["v"], v_fd, atol=3e-5 * max(1.0, np.abs(v_fd).max()))
    for j in range(len(parents)):
        qa_inv = ra["q"][j] * [1, -1, -1, -1]
        w_fd = 2 * O.quat_log(O.quat_mul(rb["q"][j], qa_inv)) / (2 * d)      # world frame
        # the difference quotient itself is off by O(d^2 |w|^3) ~ 1e-5 relative at these speeds
        np.testing.assert_allclose(r["w"][j], w_fd, atol=3e-5 * max(1.0, np.abs(w_fd).max()))


# ------------------------------------------------------------------ reward
def _ref_as_state(r):
    return r["p"].copy(), r["q"].copy(), r["v"].copy(), r["w"].copy()


def test_zero_error_reward_is_exact():
    J = 4
    parents = np.array([-1, 0, 1, 1], np.int32)
    offsets = np.array([[0, 0, 0], [0.25, 0, 0], [0, 0.5, 0], [0, 0, 0.125]], np.float32)
    skel = O.Skeleton(parents, offsets)
    quat = np.zeros((2, J, 4), np.float32)
    quat[..., 0] = 1
    clips = O.Clips(skel, [2], [30.0], np.zeros((2, 3), np.float32) + [0.5, 0.25, 1.0], quat)
    r = O.reference_state(skel, clips, 0, 0.0078125)
    e = O.error_terms(skel, clips, 0, 0.0078125, *_ref_as_state(r))
    assert np.all(e == 0.0)
    assert O.reward_from_terms(W.REWARD_MULT, e) == 1.0
    assert O.reward_from_terms(W.REWARD_FIG5, e) == float(np.float32(0.15)) + float(np.float32(0.60)) + float(np.float32(0.25))
    assert abs(O.reward_from_terms(W.REWARD_FIG5, e) - 1.0) < 1e-7
    assert abs(O.reward_from_terms(W.REWARD_ADD4, e) - 1.0) < 1e-7


def test_sim_equal_to_reference_has_tiny_error():
    sc = tiny_scene(parents=W.PARENTS_15, K=20, seed=5)
    r = O.reference_state(sc["skel"], sc["clips"], 0, 0.217)
    e = O.error_terms(sc["skel"], sc["clips"], 0, 0.217, *_ref_as_state(r))
    assert np.all(e <= 1e-10)
    assert abs(O.reward_from_terms(W.REWARD_MULT, e) - 1.0) < 1e-6


def test_error_terms_closed_forms():
    sc = tiny_scene(parents=W.PARENTS_15, K=20, seed=6)
    skel, clips, t = sc["skel"], sc["clips"], 0.3
    r = O.reference_state(skel, clips, 0, t)
    J = 15
    ee = [2, 6, 9, 12, 14]                      # bodies without children
    # (i) translate the whole character: com, body and end-effector sums follow |d|^2
    d = np.array([0.03, -0.02, 0.05])
    p, q, v, w = _ref_as_state(r)
    e = O.error_terms(skel, clips, 0, t, p + d, q, v, w)
    np.testing.assert_allclose(e, [0, 0, len(ee) * d @ d, 0, d @ d, J * d @ d, 0], atol=1e-12)
    # (ii) extra linear velocity on one body only
    p, q, v, w = _ref_as_state(r)
    v[7] += [0.1, 0.2, -0.3]
    e = O.error_terms(skel, clips, 0, t, p, q, v, w)
    np.testing.assert_allclose(e, [0, 0, 0, 0, 0, 0, 0.14], atol=1e-12)
    # (iii) extra world angular velocity on body 1 (children 2, 4, 7): its own joint velocity and
    # those of its three children each change by the same length
    p, q, v, w = _ref_as_state(r)
    dw = np.array([0.2, -0.1, 0.05])
    w[1] += dw
    e = O.error_terms(skel, clips, 0, t, p, q, v, w)
    np.testing.assert_allclose(e, [0, 4 * dw @ dw, 0, 0, 0, 0, 0], atol=1e-11)
    # (iv) turn a leaf body by eps about an arbitrary axis in its own frame: pose and ee-rot = eps^2
    p, q, v, w = _ref_as_state(r)
    eps = 0.37
    q[6] = O.quat_mul(q[6], axis_angle_quat([0.2, 0.9, -0.4], eps))
    e = O.error_terms(skel, clips, 0, t, p, q, v, w)
    # the joint velocity is expressed in the (now turned) child frame, so it turns with it
    Re = rodrigues([0.2, 0.9, -0.4], eps)
    e_vel = np.square(Re.T @ r["wl"][6] - r["wl"][6]).sum()
    np.testing.assert_allclose(e, [eps ** 2, e_vel, 0, eps ** 2, 0, 0, 0], atol=1e-11)
    # (v) turn an inner body: its own joint and each child joint see the same angle
    p, q, v, w = _ref_as_state(r)
    q[1] = O.quat_mul(axis_angle_quat([1, 2, 3], eps), q[1])
    e = O.error_terms(skel, clips, 0, t, p, q, v, w)
    np.testing.assert_allclose(e[[0, 2, 3, 4, 5, 6]], [4 * eps ** 2, 0, 0, 0, 0, 0], atol=1e-11)


def test_reward_monotone_in_injected_error():
    sc = tiny_scene(parents=W.PARENTS_15, K=20, seed=7)
    skel, clips, t = sc["skel"], sc["clips"], 0.41
    r = O.reference_state(skel, clips, 0, t)

    def run(kind, eps):
        p, q, v, w = _ref_as_state(r)
        if kind == "joint":
            q[5] = O.quat_mul(q[5], axis_angle_quat([0, 1, 0], eps))
        elif kind == "root":
            p = p + [eps, 0, 0]
        elif kind == "omega":
            w[3] += [0, 0, eps]
        elif kind == "vel":
            v[3] += [0, eps, 0]
        return O.error_terms(skel, clips, 0, t, p, q, v, w)

    # error terms that must grow, and reward presets (MULT, FIG5, ADD4) whose weight on them is non-zero
    which = dict(joint=([0], [0, 2]), root=([2, 4, 5], [0, 1, 2]), omega=([1], [0, 2]), vel=([6], [1]))
    for kind, (idx, strict) in which.items():
        prev_e, prev_r = None, None
        for eps in [0.0, 0.01, 0.05, 0.2, 0.6]:
            e = run(kind, eps)
            rews = [O.reward_from_terms(cfg, e) for cfg in (W.REWARD_MULT, W.REWARD_FIG5, W.REWARD_ADD4)]
            if prev_e is not None:
                assert np.all(e[idx] > prev_e[idx])
                assert all(rews[i] < prev_r[i] for i in strict)
                assert all(a <= b for a, b in zip(rews, prev_r))
            prev_e, prev_r = e, rews


def test_multiplicative_reward_is_product_of_factors():
    e = np.array([0.1, 3.0, 0.01, 0.2, 0.004, 0.5, 2.0])
    w = np.asarray(W.REWARD_MULT["w"], np.float32).astype(float)     # weights are fp32 parameters
    assert abs(O.reward_from_terms(W.REWARD_MULT, e) - np.prod(np.exp(-w * e))) < 1e-15


def test_fig5_preset_matches_the_printed_formula():
    """Figure 5: 0.60 exp(-4 pose) + 0.25 exp(-0.25 vel) + 0.15 exp(-8 com), done if height < 0.55 or
    reward < 0.15, with pose/vel the summed squared body position/velocity differences."""
    wl, skel, lib, pol, osk, ocl = scene_from_workload("cfg1_tiny64")
    cfg = O.make_env_config(wl.dt, 0, W.REWARD_FIG5, h_min=0.55, r_min=0.15)
    env = O.Env(osk, ocl, cfg, wl.n_envs)
    env.reset_all(0)
    clip0, t0 = env.clip_id.copy(), env.t.copy()
    sim = W.synth_sim_state(skel, lib, clip0, t0.astype(np.float64) + wl.dt, 1, wl)
    sim[2, ::7] = 0.5                                   # push some roots under 0.55 m
    out = env.step(1, sim.copy())
    J = 15
    pos, quat, lin, ang = W.split_sim(sim, J)
    m = skel["masses"].astype(float)
    n_done = 0
    for e in range(wl.n_envs):
        ref = O.reference_state(osk, ocl, clip0[e], np.float32(t0[e]) + np.float32(wl.dt))
        body_pos = pos[:, e].astype(float).reshape(J, 3)
        body_vel = lin[:, e].astype(float).reshape(J, 3)
        com_pos = (m[:, None] * body_pos).sum(0) / m.sum()
        pose_err = np.square(body_pos - ref["p"]).sum()
        vel_err = np.square(body_vel - ref["v"]).sum()
        com_err = np.square(com_pos - ref["com"]).sum()
        reward = 0.60 * math.exp(-4.0 * pose_err) + 0.25 * math.exp(-0.25 * vel_err) + 0.15 * math.exp(-8.0 * com_err)
        done = (body_pos[0, 2] < 0.55) or (reward < 0.15)
        assert abs(out["reward"][e] - reward) < 1e-7
        if abs(reward - 0.15) > 1e-6:
            assert bool(out["flags"][e] & 1) == done
        n_done += done
    assert 0 < n_done < wl.n_envs


# ------------------------------------------------------------------ flags and reset
def _rollout(name, n, steps, reward=W.REWARD_MULT, **cfg_kw):
    wl, skel, lib, pol, osk, ocl = scene_from_workload(name)
    cfg = O.make_env_config(wl.dt, wl.seed, reward, wl.h_min, **cfg_kw)
    env = O.Env(osk, ocl, cfg, n)
    obs0 = env.reset_all(0)
    hist = []

    def consume(s, sim):
        before = (env.clip_id.copy(), env.t.copy(), env.ep_len.copy())
        sim = sim.numpy()
        out = env.step(s, sim)
        hist.append(dict(before=before, after=(env.clip_id.copy(), env.t.copy(), env.ep_len.copy()),
                         sim=sim, **out))

    W.rollout_inputs(wl, skel, lib, lambda: (env.clip_id.copy(), env.t.copy()), consume, steps=steps)
    return wl, skel, lib, osk, ocl, env, obs0, hist


def test_flags_and_masked_reset_semantics():
    wl, skel, lib, osk, ocl, env, obs0, hist = _rollout("cfg5_reset_heavy", 2048, 12)
    dur = np.array([ocl.duration(c) for c in range(ocl.C)], np.float32)
    dt = np.float32(wl.dt)
    rates = []
    for h in hist:
        c0, t0, l0 = h["before"]
        c1, t1, l1 = h["after"]
        t_adv = (t0 + dt).astype(np.float32)
        term = h["sim"][2] < np.float32(wl.h_min)
        trunc = (t_adv + dt).astype(np.float32) > dur[c0]
        np.testing.assert_array_equal(h["flags"], term.astype(np.uint8) | (trunc.astype(np.uint8) << 1))
        keep = h["flags"] == 0
        # untouched envs: same clip, time advanced by exactly one fp32 add, episode length + 1
        np.testing.assert_array_equal(c1[keep], c0[keep])
        np.testing.assert_array_equal(t1[keep].view(np.uint32), t_adv[keep].view(np.uint32))
        np.testing.assert_array_equal(l1[keep], l0[keep] + 1)
        # reset envs: fresh episode somewhere that leaves at least one step
        assert np.all(l1[~keep] == 0)
        assert np.all((c1[~keep] >= 0) & (c1[~keep] < ocl.C))
        assert np.all((t1[~keep] >= 0) & (t1[~keep] < dur[c1[~keep]] - dt + 1e-6))
        rates.append(1 - keep.mean())
    assert 0.08 < np.mean(rates) < 0.35          # the reset-heavy workload resets 10-30 % per step


def test_reset_draws_are_uniform():
    wl, skel, lib, pol, osk, ocl = scene_from_workload("cfg3_16384_lib32")
    cfg = O.make_env_config(wl.dt, 12345, W.REWARD_MULT, wl.h_min)
    n = 200000
    env = O.Env(osk, ocl, cfg, n)
    env.reset_all(0)
    counts = np.bincount(env.clip_id, minlength=ocl.C)
    assert scipy.stats.chisquare(counts).pvalue > 1e-4
    dur = np.array([ocl.duration(c) for c in range(ocl.C)], np.float32)
    u = env.t / (dur[env.clip_id] - np.float32(wl.dt))
    assert u.min() >= 0 and u.max() < 1
    assert scipy.stats.kstest(u, "uniform").pvalue > 1e-4
    # the draw is a pure function of (seed, env, step): a second call agrees, another step does not
    c, t = O.reset_draw(ocl, cfg, 77, 0)
    assert (c, t) == (env.clip_id[77], env.t[77])
    assert O.reset_draw(ocl, cfg, 77, 1) != (c, t)


def test_reset_draw_from_the_published_philox_words():
    """Hand case on the first known-answer vector (counter 0, key 0 = env 0, step 0, seed 0): the clip comes from
    word 0 by the high half of a 32 x 32 multiply, the phase from the top 24 bits of word 1."""
    with open(os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")) as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    assert rows[0][:6] == ["00000000"] * 6
    x0, x1 = int(rows[0][6], 16), int(rows[0][7], 16)
    wl, skel, lib, pol, osk, ocl = scene_from_workload("cfg3_16384_lib32")
    cfg = O.make_env_config(wl.dt, 0, W.REWARD_MULT, wl.h_min)
    clip = (x0 * ocl.C) >> 32
    u = np.float32((x1 >> 8) * 2.0 ** -24)
    span = np.float32(np.float32(ocl.duration(clip)) - np.float32(wl.dt))
    t = np.float32(u * span)
    c, tt = O.reset_draw(ocl, cfg, 0, 0)
    assert c == clip == 12 and tt.view(np.uint32) == t.view(np.uint32)      # 0x6627e8d5 * 32 >> 32 = 12
    # a draw that took both from word 0, or swapped the words, would give another pair
    assert (x1 * ocl.C) >> 32 != clip and np.float32((x0 >> 8) * 2.0 ** -24) != u


def test_reset_clip_and_phase_are_jointly_uniform():
    """2-D chi-square over (clip, phase decile) of a million draws: uniform marginals alone would also pass
    if clip and phase came from the same Philox word; the joint table does not."""
    J = 1
    lib = W.make_clip_library(J, 32, (60, 600), 30.0, seed=3)
    osk = O.Skeleton([-1], np.zeros((1, 3), np.float32))
    ocl = O.Clips(osk, lib["n_frames"], lib["fps"], lib["root_pos"], lib["local_quat"])
    dt = 1.0 / 30.0
    cfg = O.make_env_config(dt, 2024, W.REWARD_MULT, 0.0)
    n = 1000000
    env = O.Env(osk, ocl, cfg, n)
    env.reset_all(0)
    dur = np.array([ocl.duration(c) for c in range(ocl.C)], np.float32)
    u = env.t / (dur[env.clip_id] - np.float32(dt))
    decile = np.minimum((u * 10).astype(np.int64), 9)
    table = np.bincount(env.clip_id.astype(np.int64) * 10 + decile, minlength=320).reshape(32, 10)
    assert table.sum() == n
    assert scipy.stats.chisquare(table.ravel()).pvalue > 1e-4                       # all 320 cells equally likely
    assert scipy.stats.chi2_contingency(table)[1] > 1e-4                            # clip independent of phase
    # the test has power: the same statistic on draws that reuse one word for both is hopeless
    x = np.random.default_rng(0).integers(0, 2 ** 32, n, dtype=np.uint64)
    fake = np.bincount(((x * 32) >> 32).astype(np.int64) * 10 + np.minimum(((x >> 8) * 10) >> 24, 9).astype(np.int64),
                       minlength=320).reshape(32, 10)
    assert scipy.stats.chisquare(fake.ravel()).pvalue < 1e-12


def test_forced_all_and_none_reset():
    for h_min, frac in [(10.0, 1.0), (-10.0, None)]:
        wl, skel, lib, pol, osk, ocl = scene_from_workload("cfg1_tiny64")
        cfg = O.make_env_config(wl.dt, 0, W.REWARD_MULT, h_min)
        env = O.Env(osk, ocl, cfg, 64)
        env.reset_all(0)
        sim = W.synth_sim_state(skel, lib, env.clip_id, env.t.astype(np.float64) + wl.dt, 1, wl)
        out = env.step(1, sim)
        if frac == 1.0:
            assert np.all(out["flags"] & 1) and np.all(env.ep_len == 0)
        else:
            assert np.all((out["flags"] & 1) == 0)


# ------------------------------------------------------------------ observation
def test_obs_single_body_closed_form():
    skel = O.Skeleton([-1], np.zeros((1, 3), np.float32))
    psi = 0.7
    q = axis_angle_quat([0, 0, 1], psi).astype(np.float32)
    quat = np.tile(q, (3, 1, 1)).astype(np.float32)
    root = np.array([[1.0, 2.0, 0.9], [1.5, 2.0, 0.9], [2.0, 2.0, 0.9]], np.float32)
    clips = O.Clips(skel, [3], [2.0], root, quat)       # 2 fps: 0.5 m per keyframe along x
    cfg = O.make_env_config(0.25, 0, W.REWARD_MULT, -1.0)
    env = O.Env(skel, clips, cfg, 1)
    env.reset_all(0)
    env.t[:] = 0.25
    sim = np.zeros((13, 1), np.float32)
    sim[0:3, 0] = [5.0, -3.0, 1.25]
    sim[3:7, 0] = q
    sim[7:10, 0] = [1.0, 0.0, 0.5]
    sim[10:13, 0] = [0.0, 1.0, 0.0]
    o = env.step(1, sim)["obs"][0]
    c, s = math.cos(psi), math.sin(psi)
    np.testing.assert_allclose(o[0:3], [0, 0, 1.25], atol=1e-7)
    np.testing.assert_allclose(o[3:6], [1, 0, 0], atol=1e-7)          # heading-local x axis
    np.testing.assert_allclose(o[6:9], [0, 0, 1], atol=1e-7)
    np.testing.assert_allclose(o[9:12], [c, -s, 0.5], atol=1e-7)      # world (1,0,.5) turned by -psi
    np.testing.assert_allclose(o[12:15], [s, c, 0], atol=1e-7)
    assert abs(o[15] - 0.5) < 1e-7                                    # t = 0.5 s of a 1 s clip
    # target: reference root at t + dt = 0.75 s -> x = 1.75, seen from the simulated root
    d = np.array([1.75 - 5.0, 2.0 + 3.0])
    np.testing.assert_allclose(o[16:19], [c * d[0] + s * d[1], -s * d[0] + c * d[1], 0.9], atol=1e-6)
    np.testing.assert_allclose(o[19:25], [1, 0, 0, 0, 0, 1], atol=1e-7)


def _rotate_scene_about_z(skel, lib, sim, J, ang, shift):
    """World rotation about z plus xy translation applied to the clips and the simulated state."""
    qz = axis_angle_quat([0, 0, 1], ang)
    Rz = rodrigues([0, 0, 1], ang)
    lib2 = dict(lib)
    root = lib["root_pos"].astype(float) @ Rz.T + shift
    lq = lib["local_quat"].astype(float).copy()
    lq[:, 0] = W._qmul(np.broadcast_to(qz, lq[:, 0].shape), lq[:, 0])
    lib2["root_pos"], lib2["local_quat"] = root.astype(np.float32), lq.astype(np.float32)
    pos, quat, lin, ang_v = W.split_sim(sim, J)
    n = sim.shape[1]
    out = np.empty_like(sim)
    P = pos.T.reshape(n, J, 3).astype(float) @ Rz.T + shift
    Q = W._qmul(np.broadcast_to(qz, (n, J, 4)), quat.T.reshape(n, J, 4).astype(float))
    out[0:3 * J] = P.reshape(n, 3 * J).T
    out[3 * J:7 * J] = Q.reshape(n, 4 * J).T
    out[7 * J:10 * J] = (lin.T.reshape(n, J, 3).astype(float) @ Rz.T).reshape(n, 3 * J).T
    out[10 * J:13 * J] = (ang_v.T.reshape(n, J, 3).astype(float) @ Rz.T).reshape(n, 3 * J).T
    return lib2, out


def test_obs_and_reward_invariant_to_heading_and_translation():
    wl, skel, lib, pol, osk, ocl = scene_from_workload("cfg1_tiny64")
    cfg = O.make_env_config(wl.dt, 0, W.REWARD_MULT, wl.h_min)
    env = O.Env(osk, ocl, cfg, 64)
    env.reset_all(0)
    st = (env.clip_id.copy(), env.t.copy(), env.ep_len.copy())
    sim = W.synth_sim_state(skel, lib, env.clip_id, env.t.astype(np.float64) + wl.dt, 1, wl)
    a = env.step(1, sim.copy())
    lib2, sim2 = _rotate_scene_about_z(skel, lib, sim, 15, 2.1, np.array([3.0, -7.0, 0.0]))
    ocl2 = O.Clips(osk, lib2["n_frames"], lib2["fps"], lib2["root_pos"], lib2["local_quat"])
    env2 = O.Env(osk, ocl2, cfg, 64)
    env2.clip_id[:], env2.t[:], env2.ep_len[:] = st
    b = env2.step(1, sim2)
    np.testing.assert_allclose(b["obs"], a["obs"], atol=2e-5)      # inputs were rounded to fp32
    np.testing.assert_allclose(b["reward"], a["reward"], atol=1e-5)
    np.testing.assert_allclose(b["terms"], a["terms"], rtol=1e-4, atol=1e-5)


def test_obs_structure():
    wl, skel, lib, osk, ocl, env, obs0, hist = _rollout("cfg1_tiny64", 64, 3)
    J = 15
    for obs in [obs0] + [h["obs"] for h in hist]:
        body = obs[:, :15 * J].reshape(-1, J, 15)
        tgt = obs[:, 15 * J + 1:].reshape(-1, J, 9)
        for tan, nrm in [(body[..., 3:6], body[..., 6:9]), (tgt[..., 3:6], tgt[..., 6:9])]:
            np.testing.assert_allclose(np.linalg.norm(tan, axis=-1), 1, atol=1e-6)
            np.testing.assert_allclose(np.linalg.norm(nrm, axis=-1), 1, atol=1e-6)
            np.testing.assert_allclose((tan * nrm).sum(-1), 0, atol=1e-6)
        np.testing.assert_allclose(body[:, 0, 0:2], 0, atol=1e-12)       # root at the origin in xy
        np.testing.assert_allclose(body[:, 0, 4], 0, atol=1e-9)          # root x-axis has no local y
        assert np.all(body[:, 0, 3] > 0)
        ph = obs[:, 15 * J]
        assert np.all((ph >= 0) & (ph <= 1))
        assert obs.shape[1] == 361


def test_obs_static_clip_target_equals_pose():
    sc = tiny_scene(parents=W.PARENTS_15, K=10, seed=9, static=True)
    cfg = O.make_env_config(1 / 30, 0, W.REWARD_MULT, -1.0)
    env = O.Env(sc["skel"], sc["clips"], cfg, 8)
    obs = env.reset_all(0)
    J = 15
    body = obs[:, :15 * J].reshape(-1, J, 15)
    tgt = obs[:, 15 * J + 1:].reshape(-1, J, 9)
    np.testing.assert_allclose(tgt, body[..., :9], atol=1e-9)
    np.testing.assert_allclose(body[..., 9:], 0, atol=1e-9)


def test_reset_env_observes_the_reference_state():
    """A reset env's observation is that of the reference pose at its new phase (sim ignored)."""
    wl, skel, lib, pol, osk, ocl = scene_from_workload("cfg1_tiny64")
    cfg = O.make_env_config(wl.dt, 0, W.REWARD_MULT, 10.0, write_back_reset=True)   # everyone terminates
    env = O.Env(osk, ocl, cfg, 64)
    env.reset_all(0)
    sim = W.synth_sim_state(skel, lib, env.clip_id, env.t.astype(np.float64) + wl.dt, 1, wl)
    out = env.step(1, sim)
    cfg2 = O.make_env_config(wl.dt, 0, W.REWARD_MULT, -10.0)
    env2 = O.Env(osk, ocl, cfg2, 64)
    env2.clip_id[:] = env.clip_id
    env2.t[:] = (env.t - np.float32(wl.dt)).astype(np.float32)
    ok = (env2.t + np.float32(wl.dt)).astype(np.float32) == env.t       # where fp32 round trips
    assert ok.sum() > 16
    # `sim` now holds the written-back reference states; feed them as the simulated state
    out2 = env2.step(2, sim)
    np.testing.assert_allclose(out2["obs"][ok], out["obs"][ok], atol=2e-5)
    assert np.all(out2["terms"][:, ok] < 1e-9)


# ------------------------------------------------------------------ policy and sampling
def test_mlp_against_torch_linear():
    import torch
    rng = np.random.default_rng(0)
    dims = (37, 64, 48, 9)
    Ws = [rng.standard_normal((o, i)).astype(np.float32) / math.sqrt(i) for i, o in zip(dims[:-1], dims[1:])]
    bs = [rng.standard_normal(o).astype(np.float32) for o in dims[1:]]
    obs = rng.standard_normal((33, 40))
    out = O.policy_forward(dims, Ws, bs, 0.1, 5, 3, obs)
    h = torch.from_numpy(obs[:, :37])
    for l, (Wl, bl) in enumerate(zip(Ws, bs)):
        h = torch.nn.functional.linear(h, torch.from_numpy(Wl).double(), torch.from_numpy(bl).double())
        if l < 2:
            h = torch.relu(h)
    np.testing.assert_allclose(out["mean"], h.numpy(), atol=1e-12)
    np.testing.assert_allclose(out["action"], out["mean"] + 0.1 * out["z"], atol=1e-15)


def test_mlp_special_cases():
    dims = (6, 5, 4)
    obs = np.arange(12, dtype=float).reshape(2, 6) - 4
    Wz = [np.zeros((5, 6), np.float32), np.zeros((4, 5), np.float32)]
    bs = [np.array([1, -2, 3, -4, 5], np.float32), np.array([0.5, 1.5, -2.5, 3.5], np.float32)]
    out = O.policy_forward(dims, Wz, bs, 0.2, 0, 0, obs)
    np.testing.assert_array_equal(out["mean"], np.tile(bs[1].astype(float), (2, 1)))     # zero weights -> bias
    W1 = np.zeros((5, 6), np.float32)
    W1[np.arange(5), np.arange(5)] = 1                                                  # [I 0]
    W2 = np.zeros((4, 5), np.float32)
    W2[np.arange(4), np.arange(4)] = 1
    zb = [np.zeros(5, np.float32), np.zeros(4, np.float32)]
    out = O.policy_forward(dims, [W1, W2], zb, 0.2, 0, 0, obs)
    np.testing.assert_array_equal(out["mean"], np.maximum(obs[:, :4], 0))                # relu kills negatives


def test_action_noise_moments_and_box_muller_geometry():
    z = np.concatenate([O.action_noise(7, e, 3, 28) for e in range(40000)])
    n = z.size
    assert abs(z.mean()) < 4 / math.sqrt(n)
    assert abs(z.var() - 1) < 4 * math.sqrt(2 / n)
    assert abs(scipy.stats.kurtosis(z, fisher=False) - 3) < 4 * math.sqrt(24 / n)
    assert scipy.stats.kstest(z[:200000], "norm").pvalue > 1e-4
    # first pair of a block: radius and angle come from the first two Philox words
    x = O.philox([11, 5, 1, 2], [7, 0])
    zz = O.action_noise(7, 11, 5, 12)[8:12]
    u1 = ((int(x[0]) >> 8) + 1) / 2 ** 24
    u2 = (int(x[1]) >> 8) / 2 ** 24
    assert abs(zz[0] ** 2 + zz[1] ** 2 + 2 * math.log(u1)) < 1e-12
    assert abs((math.atan2(zz[1], zz[0]) % (2 * math.pi)) - 2 * math.pi * u2) < 1e-12
    u3 = ((int(x[2]) >> 8) + 1) / 2 ** 24
    assert abs(zz[2] ** 2 + zz[3] ** 2 + 2 * math.log(u3)) < 1e-12
    # A not a multiple of four: the prefix of the same stream
    np.testing.assert_array_equal(O.action_noise(7, 11, 5, 69)[:28], O.action_noise(7, 11, 5, 28))


def test_logp_is_the_gaussian_log_density():
    rng = np.random.default_rng(1)
    dims = (8, 16, 5)
    Ws = [rng.standard_normal((16, 8)).astype(np.float32), rng.standard_normal((5, 16)).astype(np.float32)]
    bs = [np.zeros(16, np.float32), np.zeros(5, np.float32)]
    out = O.policy_forward(dims, Ws, bs, 0.3, 9, 2, rng.standard_normal((7, 8)))
    want = scipy.stats.norm.logpdf(out["action"], loc=out["mean"], scale=0.3).sum(axis=1)
    np.testing.assert_allclose(out["logp"], want, atol=1e-10)
    # one standard deviation per action dimension, exp(log_std)
    log_std = np.array([-2.0, -1.5, 0.0, 0.3, -0.7], np.float32)
    out2 = O.policy_forward(dims, Ws, bs, 0.3, 9, 2, rng.standard_normal((7, 8)), log_std=log_std)
    want2 = scipy.stats.norm.logpdf(out2["action"], loc=out2["mean"], scale=np.exp(log_std.astype(np.float64))).sum(axis=1)
    np.testing.assert_allclose(out2["logp"], want2, atol=1e-10)
    np.testing.assert_allclose(out2["action"] - out2["mean"], np.exp(log_std.astype(np.float64)) * out2["z"], atol=1e-14)
    same = O.policy_forward(dims, Ws, bs, 0.3, 9, 2, np.zeros((3, 8)), log_std=np.full(5, math.log(0.3), np.float32))
    ref = O.policy_forward(dims, Ws, bs, 0.3, 9, 2, np.zeros((3, 8)))
    np.testing.assert_allclose(same["action"], ref["action"], atol=1e-7)      # log 0.3 is rounded to fp32


def test_oracle_bf16_rounding_matches_torch():
    import torch
    x = np.concatenate([np.random.default_rng(3).standard_normal(2000) * 10.0 ** np.random.default_rng(4).integers(-6, 6, 2000),
                        [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895313892515355e38]])
    want = torch.from_numpy(x).float().to(torch.bfloat16).double().numpy()
    got = np.array([O.round_bf16(v) for v in x])
    np.testing.assert_array_equal(got, want)


def test_mlp_with_bf16_operands_against_torch():
    """Same chain with every layer input rounded to bf16 by torch, accumulated in fp64."""
    import torch
    rng = np.random.default_rng(5)
    dims = (37, 64, 48, 9)
    Ws = [W.round_to_bf16(rng.standard_normal((o, i)).astype(np.float32) / math.sqrt(i))[0]
          for i, o in zip(dims[:-1], dims[1:])]
    bs = [rng.standard_normal(o).astype(np.float32) for o in dims[1:]]
    obs = rng.standard_normal((33, 37)) * 3
    out = O.policy_forward(dims, Ws, bs, 0.1, 5, 3, obs, bf16_operands=True)
    h = torch.from_numpy(obs)
    for l, (Wl, bl) in enumerate(zip(Ws, bs)):
        h = h.float().to(torch.bfloat16).double()
        h = torch.nn.functional.linear(h, torch.from_numpy(Wl).double(), torch.from_numpy(bl).double())
        if l < 2:
            h = torch.relu(h)
    np.testing.assert_allclose(out["mean"], h.numpy(), atol=1e-12)
    plain = O.policy_forward(dims, Ws, bs, 0.1, 5, 3, obs)
    assert 1e-5 < np.abs(plain["mean"] - out["mean"]).max() < 0.2      # rounding matters, but only a little


def test_bf16_rounding_helper():
    import torch
    x = np.random.default_rng(0).standard_normal(1000).astype(np.float32)
    vals, bits = W.round_to_bf16(x)
    ref = torch.from_numpy(x).to(torch.bfloat16)
    np.testing.assert_array_equal(vals, ref.float().numpy())
    np.testing.assert_array_equal(bits, ref.view(torch.int16).numpy().view(np.uint16))
