"""Pins of the jerk-minimising interpolation oracle (CPU only)."""
import numpy as np
from scipy.interpolate import CubicSpline, PchipInterpolator
from scipy.optimize import minimize

from oracle.average import average_rollouts
from oracle.jmt import average_rollouts_jmt, interpolate_rollout, jerk_minimizing_curve, output_times


def _waypoints(seed, W):
    g = np.random.default_rng(seed)
    return np.cumsum(g.normal([4.0, 0.3], [1.5, 0.8], size=(W, 2)), axis=0)


def _jerk_integral(curve, t_end, n=20001):
    t = np.linspace(0.0, t_end, n)
    j = curve.derivative(3)(t)
    return float(np.trapezoid((j ** 2).sum(axis=1), t))


def test_output_times_and_knots():
    assert np.allclose(output_times(5, 20), np.arange(1, 21) * 0.25)
    assert np.allclose(output_times(10, 10), np.arange(1, 11))
    wp = _waypoints(0, 5)
    out = interpolate_rollout(wp, 20)
    # every fourth output is a decoded waypoint again, and the curve starts at the origin
    np.testing.assert_allclose(out[3::4], wp, rtol=0, atol=1e-11)
    np.testing.assert_allclose(jerk_minimizing_curve(wp)(0.0), [0.0, 0.0], atol=1e-12)
    # W outputs for W waypoints: the waypoints themselves
    np.testing.assert_allclose(interpolate_rollout(wp, 5), wp, rtol=0, atol=1e-11)


def test_motion_without_jerk_is_reproduced_exactly():
    # constant acceleration from the origin has zero jerk: the minimiser is that motion itself
    t = np.arange(1, 6, dtype=np.float64)
    wp = np.stack([3.0 * t + 0.4 * t ** 2, -0.5 * t + 0.05 * t ** 2], axis=1)
    to = output_times(5, 20)
    ref = np.stack([3.0 * to + 0.4 * to ** 2, -0.5 * to + 0.05 * to ** 2], axis=1)
    np.testing.assert_allclose(interpolate_rollout(wp, 20), ref, rtol=0, atol=1e-10)


def test_no_other_interpolant_has_less_jerk():
    for W in (5, 10):
        wp = _waypoints(W, W)
        best = jerk_minimizing_curve(wp)
        base = _jerk_integral(best, W)
        t = np.arange(W + 1.0)
        y = np.vstack([np.zeros((1, 2)), wp])
        # other smooth curves through the same knots
        rivals = [CubicSpline(t, y, bc_type="natural"), CubicSpline(t, y, bc_type="not-a-knot")]
        for r in rivals:
            tt = np.linspace(0, W, 20001)
            # a cubic spline's third derivative is piecewise constant: integrate it as such
            j = r.derivative(3)(tt[:-1] + 0.5 * (tt[1] - tt[0]))
            assert float(((j ** 2).sum(axis=1) * (tt[1] - tt[0])).sum()) > base * 1.05
        # and the minimiser plus any smooth bump that vanishes at the knots
        for k in range(3):
            bump = lambda s, k=k: np.sin(np.pi * s)[:, None] ** 6 * np.array([0.3, -0.2]) * (1 + k)
            tt = np.linspace(0, W, 40001)
            h = tt[1] - tt[0]
            curve = best(tt) + bump(tt)
            j3 = np.diff(curve, n=3, axis=0) / h ** 3
            j3_best = np.diff(best(tt), n=3, axis=0) / h ** 3
            assert (j3 ** 2).sum() * h > (j3_best ** 2).sum() * h * 1.001


def test_matches_a_brute_force_minimisation_of_the_discretised_jerk():
    # the variational definition itself, discretised: minimise the sum of squared third differences
    # over curves on a fine grid that pass through the knots
    W, per = 4, 8
    wp = _waypoints(3, W)[:, 0]
    n = W * per + 1
    knot_idx = np.arange(0, n, per)
    free = np.setdiff1d(np.arange(n), knot_idx)
    fixed_vals = np.r_[0.0, wp]
    D = np.zeros((n - 3, n))
    for i in range(n - 3):
        D[i, i:i + 4] = [-1.0, 3.0, -3.0, 1.0]
    # quadratic: solve the normal equations on the free grid points
    A = D[:, free]
    b = -D[:, knot_idx] @ fixed_vals
    x_free = np.linalg.lstsq(A, b, rcond=None)[0]
    grid = np.zeros(n)
    grid[knot_idx] = fixed_vals
    grid[free] = x_free
    curve = jerk_minimizing_curve(np.stack([wp, np.zeros(W)], axis=1))
    exact = curve(np.linspace(0, W, n))[:, 0]
    assert np.max(np.abs(grid - exact)) < 2e-2 * np.max(np.abs(wp))      # discretisation error only
    assert np.max(np.abs(grid - exact)) > 0                              # (not the same computation)
    # a cubic spline through the same knots is further away than the discretisation error
    cub = CubicSpline(np.arange(W + 1.0), fixed_vals, bc_type="natural")(np.linspace(0, W, n))
    assert np.max(np.abs(cub - exact)) > np.max(np.abs(grid - exact))


def test_interpolation_and_averaging_commute_and_reduce_to_the_plain_mean():
    g = np.random.default_rng(7)
    traj = np.stack([_waypoints(s, 5) for s in range(6)])
    a = average_rollouts_jmt(traj, 20)
    b = interpolate_rollout(average_rollouts(traj), 20)                 # linear in the waypoints
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-10)
    np.testing.assert_allclose(average_rollouts_jmt(traj, 5), average_rollouts(traj), rtol=0, atol=1e-10)
    np.testing.assert_allclose(average_rollouts_jmt(traj[:1], 20), interpolate_rollout(traj[0], 20), atol=1e-12)
    perm = g.permutation(6)
    np.testing.assert_allclose(average_rollouts_jmt(traj[perm], 20), a, rtol=0, atol=1e-10)
