"""Jerk-minimising interpolation of rollout trajectories before averaging (test infrastructure).

Sec. 3.4, trajectory averaging: every rollout's trajectory is "interpolated to 20 waypoints via
Jerk-Minimizing Trajectory fitting" and the interpolants are averaged with equal weights.  The
paper gives no formula.  The reading used by this repository (parity with the paper is therefore
unpinned; what is pinned is this reading):

  * the knots are the origin of the vehicle frame, (0, 0) at t = 0, followed by the W decoded
    waypoints at t = 1 .. W (one waypoint period apart);
  * x(t) and y(t) are, independently, the curve through the knots that minimises the integral of
    the squared jerk, int |x'''(t)|^2 dt.  That minimiser is the natural quintic spline: piecewise
    quintic, four times continuously differentiable, with x''' = x'''' = 0 at both ends;
  * the output waypoints are taken at t_j = (j + 1) W / W_out, j = 0 .. W_out - 1 (every 0.25 s for
    5 waypoints over 5 s and 20 outputs).

The spline itself comes from a library routine (scipy's B-spline interpolation with the two
end conditions); the tests pin it to the variational definition.
"""
import numpy as np
from scipy.interpolate import make_interp_spline


def output_times(n_waypoints, n_out):
    return (np.arange(n_out, dtype=np.float64) + 1.0) * n_waypoints / n_out


def jerk_minimizing_curve(waypoints):
    """waypoints: [W, 2] -> callable t -> [len(t), 2]: the natural quintic spline through
    (0, 0) at t = 0 and waypoint k at t = k + 1."""
    wp = np.asarray(waypoints, dtype=np.float64)
    knots_t = np.arange(wp.shape[0] + 1, dtype=np.float64)
    knots_y = np.vstack([np.zeros((1, 2)), wp])
    natural = [(3, np.zeros(2)), (4, np.zeros(2))]
    return make_interp_spline(knots_t, knots_y, k=5, bc_type=(natural, natural))


def interpolate_rollout(waypoints, n_out):
    """[W, 2] -> [n_out, 2] float64."""
    wp = np.asarray(waypoints, dtype=np.float64)
    return jerk_minimizing_curve(wp)(output_times(wp.shape[0], n_out))


def average_rollouts_jmt(traj, n_out):
    """traj: [N, W, 2] -> [n_out, 2]: every rollout interpolated, then the equal-weight mean
    (in that order, as the paper states it)."""
    traj = np.asarray(traj, dtype=np.float64)
    out = np.zeros((n_out, 2), dtype=np.float64)
    for i in range(traj.shape[0]):
        out += interpolate_rollout(traj[i], n_out)
    return out / traj.shape[0]
