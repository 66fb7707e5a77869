"""Philox4x32-10 counter-based generator and the Gumbel noise built on it.

Test infrastructure (CPU oracle).  The paper only says that the trajectory
section is sampled at non-zero temperature with independent draws per rollout
(Sec. 3.4, "Trajectory-only stochasticity" / "Shared prefix"); it names no
generator.  The reading used by this repository: Philox4x32 with 10 rounds
(Salmon, Moraes, Dror, Shaw, "Parallel random numbers: as easy as 1, 2, 3",
SC'11), keyed by the rollout's 64-bit seed, with the counter made of the
vocabulary index, the position inside the block, the denoising step and the
block index, so that a draw depends on nothing but (seed, block, step,
position, vocabulary id).  Each uniform is assembled from two streams: an 8-bit
coarse value (16 ids per Philox block) and 23 fine bits (4 ids per block).

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


FINE_STREAM = 1 << 31   # added to the position word of the counter for the second stream


def uniform_from_parts(coarse, fine):
    """Map an 8-bit coarse value and a 23-bit fine value to the open interval (0, 1).

    u = (coarse + (fine + 0.5) * 2**-23) / 256: the coarse byte picks one of 256
    equal bins, the fine bits a point inside it, centred in its sub-bin.  u is a
    multiple of 2**-32 in [2**-32, 1 - 2**-32], so -ln(-ln(u)) is always finite
    (between -3.1 and 22.2).
    """
    coarse = np.asarray(coarse, dtype=np.float64)
    fine = np.asarray(fine, dtype=np.float64)
    return (coarse + (fine + 0.5) * (2.0 ** -23)) / 256.0


def coarse_bytes(seed, block_idx, step, position, vocab):
    """The coarse byte of every vocabulary id of one row: id v takes byte v % 16
    (little-endian inside the four output words) of the Philox block with
    counter (v // 16, position, step, block_idx)."""
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    nctr = (vocab + 15) // 16
    ctr = np.arange(nctr, dtype=np.uint64)
    w = philox4x32_vec(ctr, np.uint64(position), np.uint64(step), np.uint64(block_idx),
                       seed & MASK32, seed >> 32)
    words = np.stack(w, axis=1).reshape(-1)                       # word k of block c at 4 c + k
    shifts = np.array([0, 8, 16, 24], dtype=np.uint64)
    return ((words[:, None] >> shifts[None, :]) & np.uint64(0xFF)).reshape(-1)[:vocab]


def fine_bits(seed, block_idx, step, position, vocab):
    """The 23 fine bits of every vocabulary id of one row: id v takes the top 23
    bits of word v % 4 of the Philox block with counter
    (v // 4, position + 2**31, step, block_idx) (a second stream: the position
    word never reaches 2**31 otherwise)."""
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    nctr = (vocab + 3) // 4
    ctr = np.arange(nctr, dtype=np.uint64)
    w = philox4x32_vec(ctr, np.uint64(position + FINE_STREAM), np.uint64(step), np.uint64(block_idx),
                       seed & MASK32, seed >> 32)
    words = np.stack(w, axis=1).reshape(-1)[:vocab]
    return words >> np.uint64(9)


def gumbel_row(seed, block_idx, step, position, vocab):
    """Standard Gumbel noise g[v] = -ln(-ln(u[v])) for one row of a block, with
    u[v] = uniform_from_parts(coarse byte of v, fine bits of v).  A draw depends
    on nothing but (seed, block, step, position, vocabulary id).

    The uniform is split in two so that an implementation can bound a draw from
    its coarse byte alone (one Philox block per 16 ids) and spend the second
    Philox block only on the few ids whose bound can still win the arg-max.
    """
    u = uniform_from_parts(coarse_bytes(seed, block_idx, step, position, vocab),
                           fine_bits(seed, block_idx, step, position, vocab))
    return -np.log(-np.log(u))
