"""Philox4x32-10 counter-based generator and the Gumbel noise built on it.

Test infrastructure (CPU oracle).  The paper only says that the trajectory
section is sampled at non-zero temperature with independent draws per rollout
(Sec. 3.4, "Trajectory-only stochasticity" / "Shared prefix"); it names no
generator.  The reading used by this repository: Philox4x32 with 10 rounds
(Salmon, Moraes, Dror, Shaw, "Parallel random numbers: as easy as 1, 2, 3",
SC'11), keyed by the rollout's 64-bit seed, with the counter made of the
vocabulary index, the position inside the block, the denoising step and the
block index, so that a draw depends on nothing but (seed, block, step,
position, vocabulary id).

Two implementations live here on purpose: a scalar one on Python integers that
follows the published round function literally, and a numpy one used for whole
rows.  The tests pin the scalar one to the published known-answer values and
the vectorised one to the scalar one.
"""
import numpy as np

PHILOX_M0 = 0xD2511F53
PHILOX_M1 = 0xCD9E8D57
PHILOX_W0 = 0x9E3779B9  # golden ratio
PHILOX_W1 = 0xBB67AE85  # sqrt(3) - 1
MASK32 = 0xFFFFFFFF


def philox4x32_scalar(counter, key, rounds=10):
    """One Philox4x32 block on Python ints.

    counter: 4 words, key: 2 words (each 0 <= w < 2**32).  Returns 4 words.
    Round: (c0, c1, c2, c3) -> (hi(M1*c2) ^ c1 ^ k0, lo(M1*c2),
                                hi(M0*c0) ^ c3 ^ k1, lo(M0*c0));
    the key is bumped by the Weyl constants between rounds.
    """
    c0, c1, c2, c3 = (int(w) & MASK32 for w in counter)
    k0, k1 = (int(w) & MASK32 for w in key)
    for r in range(rounds):
        if r > 0:
            k0 = (k0 + PHILOX_W0) & MASK32
            k1 = (k1 + PHILOX_W1) & MASK32
        p0 = PHILOX_M0 * c0
        p1 = PHILOX_M1 * c2
        hi0, lo0 = p0 >> 32, p0 & MASK32
        hi1, lo1 = p1 >> 32, p1 & MASK32
        c0, c1, c2, c3 = (hi1 ^ c1 ^ k0) & MASK32, lo1, (hi0 ^ c3 ^ k1) & MASK32, lo0
    return (c0, c1, c2, c3)


def philox4x32_vec(c0, c1, c2, c3, k0, k1, rounds=10):
    """Vectorised Philox4x32 on numpy uint64 arrays holding 32-bit words."""
    c0 = np.asarray(c0, dtype=np.uint64) & np.uint64(MASK32)
    c1 = np.asarray(c1, dtype=np.uint64) & np.uint64(MASK32)
    c2 = np.asarray(c2, dtype=np.uint64) & np.uint64(MASK32)
    c3 = np.asarray(c3, dtype=np.uint64) & np.uint64(MASK32)
    c0, c1, c2, c3 = np.broadcast_arrays(c0, c1, c2, c3)
    k0 = np.uint64(int(k0) & MASK32)
    k1 = np.uint64(int(k1) & MASK32)
    m32 = np.uint64(MASK32)
    s32 = np.uint64(32)
    for r in range(rounds):
        if r > 0:
            k0 = (k0 + np.uint64(PHILOX_W0)) & m32
            k1 = (k1 + np.uint64(PHILOX_W1)) & m32
        p0 = np.uint64(PHILOX_M0) * c0
        p1 = np.uint64(PHILOX_M1) * c2
        hi0, lo0 = p0 >> s32, p0 & m32
        hi1, lo1 = p1 >> s32, p1 & m32
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
    return c0, c1, c2, c3


def uniform_from_word(x):
    """Map a 32-bit word to the open interval (0, 1).

    u = ((x >> 9) + 0.5) * 2**-23: the top 23 bits, centred in their bin.  Every
    value is exactly representable in fp32 as well as fp64 (24 significant
    bits), lies in [2**-24, 1 - 2**-24], and so -ln(-ln(u)) is always finite.
    """
    x = np.asarray(x, dtype=np.uint64)
    return ((x >> np.uint64(9)).astype(np.float64) + 0.5) * (2.0 ** -23)


def gumbel_row(seed, block_idx, step, position, vocab):
    """Standard Gumbel noise g[v] = -ln(-ln(u[v])) for one row of a block.

    Counter = (v // 4, position, step, block_idx), key = (seed low word, seed
    high word); vocabulary id v takes output word v % 4 of its counter.
    """
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    nctr = (vocab + 3) // 4
    ctr = np.arange(nctr, dtype=np.uint64)
    w = philox4x32_vec(ctr, np.uint64(position), np.uint64(step), np.uint64(block_idx),
                       seed & MASK32, seed >> 32)
    words = np.stack(w, axis=1).reshape(-1)[:vocab]
    u = uniform_from_word(words)
    return -np.log(-np.log(u))
