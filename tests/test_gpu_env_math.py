"""The env kernel's approximations in isolation (im_debug_math) against fp64 closed forms.

The kernel avoids inverse trigonometry where angles are small: the squared geodesic angle comes from an
arcsine series on sin^2(theta / 2) up to 0.15 (atan2 beyond), slerp is q0 exp(alpha h) with Taylor polynomials
for cos and sin(x)/x up to |h| = 0.5 (sincos beyond).  Both branches and both sides of each switch point are
swept here; the bound is the one a single observation or error-term entry gets (1e-5 + 1e-4 relative), with the
1e-6 that one factor of a 9-link chain may use for the interpolated quaternion."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2609_09821_b200 import binding as B

pytestmark = pytest.mark.gpu


def _unit(rng, n, k):
    v = rng.standard_normal((n, k))
    return v / np.linalg.norm(v, axis=1, keepdims=True)


def test_squared_angle_over_both_branches_and_the_switch_point():
    rng = np.random.default_rng(0)
    # rotation angles from 0 to pi, dense around the switch at sin^2(theta/2) = 0.15 (theta = 0.7954 rad)
    theta_sw = 2 * np.arcsin(np.sqrt(0.15))
    theta = np.concatenate([np.linspace(0, np.pi, 4001), theta_sw + np.linspace(-1e-3, 1e-3, 2001),
                            10.0 ** np.linspace(-8, -2, 500)])
    axis = _unit(rng, len(theta), 3)
    scale = rng.uniform(0.5, 2.0, len(theta))             # the function takes quaternions of any norm ...
    sign = rng.choice([-1.0, 1.0], len(theta))            # ... and either sign
    q = np.concatenate([np.cos(theta / 2)[:, None], np.sin(theta / 2)[:, None] * axis], axis=1) * (scale * sign)[:, None]
    got = B.debug_math(B.DEBUG_ANGLE_SQ, torch.from_numpy(q.astype(np.float32)).cuda()).cpu().numpy().astype(np.float64)
    # what the fp32 inputs define, in fp64 through the oracle's geodesic angle
    q32 = q.astype(np.float32).astype(np.float64)
    want = np.array([O.geodesic_angle(x / np.linalg.norm(x)) ** 2 for x in q32])
    err = np.abs(got - want)
    assert np.all(err <= 2e-6 + 2e-6 * want), (err.max(), theta[np.argmax(err)])
    # both branches ran
    u = np.sin(theta / 2) ** 2
    assert (u <= 0.15).sum() > 1000 and (u > 0.15).sum() > 1000


def test_slerp_over_both_branches_and_the_switch_point():
    rng = np.random.default_rng(1)
    # half-angle |h| from 0 to just under pi/2 (the shortest arc never exceeds it; at exactly pi/2 both arcs are
    # equally short and the reference may take the other one), dense around the switch at 0.5
    th = np.concatenate([np.linspace(0, np.pi / 2 - 1e-3, 3001), 0.5 + np.linspace(-1e-3, 1e-3, 1001), 10.0 ** np.linspace(-8, -2, 300)])
    n = len(th)
    q0 = _unit(rng, n, 4).astype(np.float32)
    h = (_unit(rng, n, 3) * th[:, None]).astype(np.float32)
    alpha = rng.uniform(0, 1, n).astype(np.float32)
    alpha[:50] = 0.0
    alpha[50:100] = 1.0
    inp = np.concatenate([q0, h, alpha[:, None]], axis=1).astype(np.float32)
    out = B.debug_math(B.DEBUG_SLERP, torch.from_numpy(inp).cuda()).cpu().numpy().astype(np.float64)
    # closed form from the fp32 inputs: q1 = q0 exp(h); the oracle's slerp between q0 and q1 at alpha
    q0d = q0.astype(np.float64)
    q0d /= np.linalg.norm(q0d, axis=1, keepdims=True)
    hd = h.astype(np.float64)
    thd = np.linalg.norm(hd, axis=1)
    sinc = np.where(thd > 0, np.sin(thd) / np.where(thd > 0, thd, 1), 1.0)
    e = np.concatenate([np.cos(thd)[:, None], sinc[:, None] * hd], axis=1)
    worst = 0.0
    for i in range(n):
        q1 = O.quat_mul(q0d[i], e[i])
        want = O.slerp(q0d[i], q1, float(alpha[i]))
        got = out[i, :4] / np.linalg.norm(q0[i].astype(np.float64))      # the product keeps the norm of q0
        d = min(np.abs(got - want).max(), np.abs(got + want).max())
        worst = max(worst, d)
        # |q0| of a random fp32 unit vector is 1 to 1e-7: the product keeps that norm
    assert worst <= 1e-6, worst
    np.testing.assert_allclose(out[:, 4:], 2.0 * hd, rtol=1e-6, atol=1e-12)
    assert (thd <= 0.5).sum() > 500 and (thd > 0.5).sum() > 500
