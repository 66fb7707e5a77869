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

The definition, for vocabulary id v of one row (`exponential_scalar` is this
paragraph on Python integers, nothing else):

    group j = v // 16 has the 32-bit word
        R_j  = output word j % 4 of Philox(counter (j // 4, position, step, block))
    every id has 23 bits of its own
        f_v  = top 23 bits of output word v % 4 of
               Philox(counter (v // 4, position + 2**31, step, block))
    the id 16 j + R_j % 16 is the group's leader and holds the group's minimum
        E    = -ln(U) / 16,   U = ((R_j >> 4) + (f_leader + 0.5) 2**-23) / 2**28
    every other id of the group has
        E_v  = E_leader - ln((f_v + 0.5) 2**-23)
    and the noise is g_v = -ln(E_v).

The counters are the plain running indices of groups and ids: nothing in them
knows how an implementation walks through a row.  That the E_v are independent
Exp(1) variates (so that the g_v are independent standard Gumbel variates) is
the memorylessness of the exponential distribution, see `exponential_row`.

Three implementations live here on purpose: Philox on Python integers that
follows the published round function literally, `exponential_scalar` (the
definition above, one id at a time) and numpy versions for whole rows.  The
tests pin the scalar Philox to the published known-answer values, the
vectorised functions to the scalar ones, and the distribution of the draws to
what the construction promises.
"""
import math

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
GROUP = 16              # vocabulary ids per group


def exponential_scalar(seed, block_idx, step, position, v):
    """E[v] of a single vocabulary id on Python integers and math.log: the definition in
    the module docstring, line by line."""
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    key = (seed & MASK32, seed >> 32)

    def fine(u):
        return philox4x32_scalar((u // 4, position + FINE_STREAM, step, block_idx), key)[u % 4] >> 9

    j = v // GROUP
    R = philox4x32_scalar((j // 4, position, step, block_idx), key)[j % 4]
    leader = GROUP * j + R % GROUP
    U = ((R >> 4) + (fine(leader) + 0.5) * 2.0 ** -23) * 2.0 ** -28      # exact in fp64 (51 bits)
    e = -math.log(U) / GROUP
    if v != leader:
        e += -math.log((fine(v) + 0.5) * 2.0 ** -23)
    return e


def group_words(seed, block_idx, step, position, vocab):
    """The 32-bit word R_j of every group j (ids 16 j .. 16 j + 15) of one row:
    output word j % 4 of the Philox block with counter (j // 4, position, step,
    block_idx), i.e. the blocks 0, 1, 2, ... of the stream read word by word."""
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    ngroups = (vocab + GROUP - 1) // GROUP
    ctr = np.arange((ngroups + 3) // 4, dtype=np.uint64)
    w = philox4x32_vec(ctr, np.uint64(position), np.uint64(step), np.uint64(block_idx),
                       seed & MASK32, seed >> 32)
    return np.stack(w, axis=1).reshape(-1)[:ngroups]


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


def leader_exponential(word, fine):
    """The smallest exponential variate of a group, from the group's word and the
    fine bits of the id that holds it.

    U = (h + (f + 0.5) 2**-23) / 2**28 with h = word >> 4 is uniform on (0, 1) in
    steps of 2**-51; the minimum of 16 independent Exp(1) variates is Exp(1) / 16,
    so E = -ln(U) / 16.  Written through 1 - U, which fp64 holds exactly, so that
    the tail U -> 1 (the large Gumbel draws) loses nothing.
    """
    h = (np.asarray(word, dtype=np.uint64) >> np.uint64(4)).astype(np.float64)
    f = np.asarray(fine, dtype=np.float64)
    one_minus_u = ((2.0 ** 28 - h) - (f + 0.5) * (2.0 ** -23)) * (2.0 ** -28)
    return -np.log1p(-one_minus_u) / GROUP


def exponential_row(seed, block_idx, step, position, vocab):
    """E[v], independent Exp(1) variates for the ids of one row, as an exponential race
    per group of 16 ids:

      * the group's word R picks the id that holds the group's minimum, the
        "leader" 16 j + R % 16, and with the leader's fine bits the minimum itself
        (`leader_exponential`);
      * every other id of the group gets the minimum plus a fresh Exp(1) variate
        -ln((f + 0.5) 2**-23) from its own fine bits.

    By the memorylessness of the exponential distribution this is exactly a family
    of independent Exp(1) variates: the minimum of 16 of them is Exp(1) / 16, it sits
    at a uniformly random place, and the others exceed it by independent Exp(1)
    amounts.  What it buys an implementation: the word of a group alone bounds all
    16 draws of the group from below, so the per-id stream is needed only for the few
    ids that can still win an arg-max.
    """
    ngroups = (vocab + GROUP - 1) // GROUP
    padded = ngroups * GROUP                        # the leader of the last group may lie beyond vocab
    words = group_words(seed, block_idx, step, position, vocab)
    fine = fine_bits(seed, block_idx, step, position, padded).astype(np.float64)
    leader = np.arange(ngroups) * GROUP + (words & np.uint64(15)).astype(np.int64)
    e_min = leader_exponential(words, fine[leader])
    e = np.repeat(e_min, GROUP) - np.log((fine + 0.5) * (2.0 ** -23))
    e[leader] = e_min
    return e[:vocab]


def gumbel_row(seed, block_idx, step, position, vocab):
    """Standard Gumbel noise g[v] = -ln(E[v]) for one row of a block (E from
    `exponential_row`: -ln of an Exp(1) variate is a standard Gumbel variate).  A draw
    depends on nothing but (seed, block, step, position, vocabulary id)."""
    return -np.log(exponential_row(seed, block_idx, step, position, vocab))
