"""Equal-weight average of N rollout trajectories (test infrastructure).

Sec. 3.4, trajectory averaging: tau_out = (1/N) * sum_i tau^(i).
"""
import numpy as np


def average_rollouts(traj):
    """traj: [N, W, 2] -> [W, 2] float64 mean over the rollout axis."""
    traj = np.asarray(traj, dtype=np.float64)
    n = traj.shape[0]
    out = np.zeros(traj.shape[1:], dtype=np.float64)
    for i in range(n):
        out += traj[i]
    return out / n
