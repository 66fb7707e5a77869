"""Shared-prefix fork and private suffix append (test infrastructure).

Sec. 3.4 ("Shared prefix"): the deterministic sections are decoded once, the KV
cache is forked N times, and each rollout continues on its own.  Sec. 3.3:
finished blocks stay in the cache and are reused without recomputation.

A fork shares the prefix arrays by reference (they are never written) and owns
an initially empty suffix per layer.  Committing a block appends that rollout's
block K/V rows, bit for bit, to its suffix.
"""
import numpy as np


class ForkSet:
    """N rollouts over one shared prefix.  prefix_k/v: per-layer list of
    [P, Hkv, D] arrays of bf16 bit patterns (uint16) or floats."""

    def __init__(self, prefix_k, prefix_v, n_forks, seeds):
        assert len(prefix_k) == len(prefix_v)
        assert len(seeds) == n_forks
        self.prefix_k = list(prefix_k)
        self.prefix_v = list(prefix_v)
        self.n_forks = int(n_forks)
        self.seeds = [int(s) for s in seeds]
        n_layers = len(self.prefix_k)
        shape_tail = self.prefix_k[0].shape[1:]
        dt = self.prefix_k[0].dtype
        self.suffix_k = [[np.zeros((0,) + shape_tail, dtype=dt) for _ in range(n_forks)]
                         for _ in range(n_layers)]
        self.suffix_v = [[np.zeros((0,) + shape_tail, dtype=dt) for _ in range(n_forks)]
                         for _ in range(n_layers)]

    def suffix_len(self, f):
        return self.suffix_k[0][f].shape[0]

    def kv_commit(self, layer, k_blk, v_blk):
        """k_blk, v_blk: [N, d, Hkv, D]; rollout f's rows go to rollout f only."""
        k_blk = np.asarray(k_blk)
        v_blk = np.asarray(v_blk)
        assert k_blk.shape[0] == self.n_forks
        for f in range(self.n_forks):
            self.suffix_k[layer][f] = np.concatenate([self.suffix_k[layer][f], k_blk[f]], axis=0)
            self.suffix_v[layer][f] = np.concatenate([self.suffix_v[layer][f], v_blk[f]], axis=0)
