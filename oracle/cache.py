"""Shared-prefix fork and private suffix append (test infrastructure).

Sec. 3.4 ("Shared prefix"): the deterministic sections are decoded once, the KV
cache is forked N times, and each rollout continues on its own.  Sec. 3.3:
finished blocks stay in the cache and are reused without recomputation.

A fork shares the prefix arrays by reference (they are never written) and owns
an initially empty suffix per layer.  Committing a block appends that rollout's
block K/V rows, bit for bit, to its suffix.

The scene-level order of Sec. 3.4: a set of ONE rollout decodes the first three
(deterministic) sections; each of its finished blocks is appended to the shared
prefix itself (`extend_prefix`); then `fork` makes N rollouts over that longer
prefix, each with an empty suffix and a seed of its own.
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

    def extend_prefix(self, layer, k_blk, v_blk):
        """The one rollout of a deterministic set commits a block to the shared prefix:
        k_blk, v_blk [1, d, Hkv, D] are appended to the prefix of `layer` (a new array:
        whoever forked from the shorter prefix keeps reading that one)."""
        assert self.n_forks == 1, "only a set of one rollout extends its prefix"
        assert self.suffix_len(0) == 0, "the prefix stays in front of every private suffix"
        k_blk = np.asarray(k_blk)
        v_blk = np.asarray(v_blk)
        assert k_blk.shape[0] == 1 and v_blk.shape[0] == 1
        self.prefix_k[layer] = np.concatenate([self.prefix_k[layer], k_blk[0]], axis=0)
        self.prefix_v[layer] = np.concatenate([self.prefix_v[layer], v_blk[0]], axis=0)

    def fork(self, n_forks, seeds):
        """N rollouts over this set's current prefix (shared by reference), empty suffixes."""
        assert self.suffix_len(0) == 0
        return ForkSet(self.prefix_k, self.prefix_v, n_forks, seeds)
