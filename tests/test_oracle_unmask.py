"""Pins for the Philox/Gumbel generator and the unmasking rule of the oracle."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import MASKED, COMMITTED, SCAFFOLD
from oracle.philox import (coarse_bytes, fine_bits, gumbel_row, philox4x32_scalar, philox4x32_vec,
                           uniform_from_parts)
from oracle.unmask import unmask_step

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _kat():
    rows = []
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            w = [int(x, 16) for x in line.split()]
            rows.append((w[0:4], w[4:6], w[6:10]))
    return rows


def test_philox_known_answers():
    rows = _kat()
    assert len(rows) == 3
    for ctr, key, expect in rows:
        assert list(philox4x32_scalar(ctr, key)) == expect


def test_philox_vectorised_equals_scalar():
    g = np.random.default_rng(0)
    ctr = g.integers(0, 2 ** 32, size=(64, 4), dtype=np.uint64)
    key = (0x12345678, 0x9ABCDEF0)
    out = philox4x32_vec(ctr[:, 0], ctr[:, 1], ctr[:, 2], ctr[:, 3], key[0], key[1])
    for r in range(64):
        assert tuple(int(o[r]) for o in out) == philox4x32_scalar(ctr[r], key)
    for ctr_, key_, expect in _kat():
        out = philox4x32_vec(*[np.array([c]) for c in ctr_], key_[0], key_[1])
        assert [int(o[0]) for o in out] == expect


def test_uniform_map_is_open_interval_and_monotone():
    c = np.array([0, 0, 0, 1, 127, 128, 255, 255])
    f = np.array([0, 1, 2 ** 23 - 1, 0, 2 ** 23 - 1, 0, 0, 2 ** 23 - 1])
    u = uniform_from_parts(c, f)
    assert u[0] == 2.0 ** -32 and u[-1] == 1.0 - 2.0 ** -32
    assert np.all(np.diff(u) > 0)                      # ordered by (coarse, fine)
    assert u[3] - u[2] == 2.0 ** -31                   # bins tile (0, 1) without gap or overlap
    assert np.all(u * 2.0 ** 32 == np.round(u * 2.0 ** 32))
    g = -np.log(-np.log(u))
    assert np.all(np.isfinite(g)) and -3.1 < g[0] and g[-1] < 22.2


def test_gumbel_row_layout_and_independence_from_vocab_size():
    seed = 0xDEADBEEFCAFEF00D
    a = gumbel_row(seed, 3, 2, 5, 37)
    b = gumbel_row(seed, 3, 2, 5, 64)
    np.testing.assert_array_equal(a, b[:37])
    key = (seed & 0xFFFFFFFF, seed >> 32)
    # coarse: byte v % 16 of counter (v // 16, pos, step, block); fine: top 23 bits of word v % 4 of
    # counter (v // 4, pos + 2^31, step, block); both under key (lo, hi)
    for v in (0, 5, 18, 36):
        cw = philox4x32_scalar((v // 16, 5, 2, 3), key)[(v % 16) // 4]
        c = (cw >> (8 * (v % 4))) & 0xFF
        f = philox4x32_scalar((v // 4, 5 + 2 ** 31, 2, 3), key)[v % 4] >> 9
        u = (c + (f + 0.5) * 2.0 ** -23) / 256.0
        assert a[v] == -math.log(-math.log(u))
        assert coarse_bytes(seed, 3, 2, 5, 37)[v] == c and fine_bits(seed, 3, 2, 5, 37)[v] == f
    # every counter field and the seed matter
    for other in (gumbel_row(seed + 1, 3, 2, 5, 37), gumbel_row(seed, 4, 2, 5, 37),
                  gumbel_row(seed, 3, 1, 5, 37), gumbel_row(seed, 3, 2, 6, 37),
                  gumbel_row(seed ^ (1 << 40), 3, 2, 5, 37)):
        assert not np.array_equal(a, other)


def test_coarse_byte_bounds_the_draw():
    # what lets an implementation skip the second stream: g < -ln(-ln((c + 1) / 256)) for c < 255
    g = gumbel_row(777, 1, 4, 9, 50000)
    c = coarse_bytes(777, 1, 4, 9, 50000).astype(np.float64)
    low = c < 255
    with np.errstate(divide="ignore"):
        upper = -np.log(-np.log((c + 1.0) / 256.0))
        lower = -np.log(-np.log(c / 256.0))
    assert np.all(g[low] < upper[low]) and np.all(g[c > 0] > lower[c > 0])
    # the two streams are not the same numbers: coarse bytes are uncorrelated with the fine bits
    f = fine_bits(777, 1, 4, 9, 50000).astype(np.float64)
    assert abs(np.corrcoef(c, f)[0, 1]) < 0.02
    counts = np.bincount(c.astype(int), minlength=256)
    assert counts.min() > 120 and counts.max() < 280    # 50000 / 256 = 195 expected per bin


def test_gumbel_uniformity_ks():
    # Kolmogorov-Smirnov distance of exp(-exp(-g)) = u from U(0,1) on 2e5 draws
    g = gumbel_row(12345, 0, 0, 0, 200000)
    u = np.sort(np.exp(-np.exp(-g)))
    n = len(u)
    dist = np.max(np.abs(u - (np.arange(n) + 0.5) / n))
    assert dist < 1.63 / math.sqrt(n)          # 1 % critical value


def _mk(N, d, V, seed, scaffold=()):
    g = np.random.default_rng(seed)
    logits = g.standard_normal((N, d, V)) * 2.0
    tokens = np.full((N, d), V - 1, dtype=np.int32)
    state = np.full((N, d), MASKED, dtype=np.uint8)
    for i in scaffold:
        tokens[:, i] = 7 + i
        state[:, i] = SCAFFOLD
    return logits, tokens, state


def test_greedy_matches_library_argmax_and_softmax():
    import torch
    N, d, V = 2, 6, 50
    logits, tokens, state = _mk(N, d, V, 1, scaffold=(1, 4))
    r = unmask_step(logits, tokens, state, [1, 2], threshold=-1.0, temperature=0.0, block_idx=0, step=0)
    sm = torch.softmax(torch.from_numpy(logits), dim=-1).numpy()
    for f in range(N):
        for i in range(d):
            if i in (1, 4):
                assert r["tokens"][f, i] == 7 + i and r["state"][f, i] == SCAFFOLD
                assert np.isnan(r["conf"][f, i])
            else:
                assert r["tokens"][f, i] == int(np.argmax(logits[f, i]))
                assert r["state"][f, i] == COMMITTED
                assert abs(r["conf"][f, i] - sm[f, i].max()) < 1e-14
    assert list(r["n_committed"]) == [4, 4] and list(r["n_left"]) == [0, 0]
    assert not r["fallback"].any()


def test_threshold_rules():
    N, d, V = 1, 5, 8
    logits = np.zeros((N, d, V))
    # confidences: position i has top logit a_i -> conf = e^a / (e^a + 7)
    tops = [1.0, 4.0, 2.0, 6.0, 3.0]
    for i, a in enumerate(tops):
        logits[0, i, (3 * i) % V] = a
    conf = [math.exp(a) / (math.exp(a) + 7.0) for a in tops]
    tokens = np.full((N, d), -5, dtype=np.int32)
    state = np.zeros((N, d), dtype=np.uint8)
    # strict '>' : a threshold exactly equal to a position's confidence does not commit it
    r0 = unmask_step(logits, tokens, state, [0], threshold=0.0, temperature=0.0, block_idx=0, step=0)
    np.testing.assert_allclose(r0["conf"][0], conf, rtol=1e-14)
    r = unmask_step(logits, tokens, state, [0], threshold=float(r0["conf"][0, 1]), temperature=0.0,
                    block_idx=0, step=0)
    assert list(r["state"][0]) == [MASKED, MASKED, MASKED, COMMITTED, MASKED]
    assert r["tokens"][0, 3] == 9 % V and list(r["n_committed"]) == [1] and list(r["n_left"]) == [4]
    assert not r["fallback"][0]
    np.testing.assert_allclose(r["conf"][0], conf, rtol=1e-14)
    # threshold >= 1: exactly one commit per step, most confident first, block ends in #masked steps
    order = []
    st, tk = state, tokens
    for step in range(d):
        r = unmask_step(logits, tk, st, [0], threshold=1.0, temperature=0.0, block_idx=0, step=step)
        assert r["n_committed"][0] == 1 and r["fallback"][0]
        newly = [i for i in range(d) if st[0, i] == MASKED and r["state"][0, i] == COMMITTED]
        order += newly
        st, tk = r["state"], r["tokens"]
    assert order == [3, 1, 4, 2, 0] and not np.any(st == MASKED)
    r = unmask_step(logits, tk, st, [0], threshold=1.0, temperature=0.0, block_idx=0, step=d)
    assert r["n_committed"][0] == 0 and r["n_left"][0] == 0          # finished rollout: no-op
    np.testing.assert_array_equal(r["tokens"], tk)
    # threshold < 0: everything commits at once
    r = unmask_step(logits, tokens, state, [0], threshold=-0.5, temperature=0.0, block_idx=0, step=0)
    assert np.all(r["state"] == COMMITTED) and r["n_committed"][0] == d


def test_ties_take_lowest_index():
    logits = np.zeros((1, 3, 4))
    logits[0, :, 1] = 2.0
    logits[0, :, 3] = 2.0                      # vocabulary tie -> id 1
    tokens = np.zeros((1, 3), dtype=np.int32)
    state = np.zeros((1, 3), dtype=np.uint8)
    r = unmask_step(logits, tokens, state, [0], threshold=2.0, temperature=0.0, block_idx=0, step=0)
    # all three confidences equal -> fallback picks position 0
    assert list(r["state"][0]) == [COMMITTED, MASKED, MASKED] and r["tokens"][0, 0] == 1
    assert r["score_margin"][0, 0] == 0.0


def test_scaffold_and_committed_never_rewritten_and_progress():
    N, d, V = 3, 8, 33
    logits, tokens, state = _mk(N, d, V, 5, scaffold=(0, 3, 7))
    state[1, 2] = COMMITTED
    tokens[1, 2] = 11
    tk, st = tokens, state
    steps = 0
    while np.any(st == MASKED):
        before_t, before_s = tk.copy(), st.copy()
        r = unmask_step(logits, tk, st, [9, 9, 10], threshold=0.2, temperature=0.7, block_idx=1, step=steps)
        tk, st = r["tokens"], r["state"]
        keep = before_s != MASKED
        np.testing.assert_array_equal(tk[keep], before_t[keep])
        np.testing.assert_array_equal(st[keep], before_s[keep])
        for f in range(N):
            if np.any(before_s[f] == MASKED):
                assert r["n_committed"][f] >= 1
            assert r["n_left"][f] == np.sum(st[f] == MASKED)
        steps += 1
        assert steps <= d
    # rollouts 0 and 1 share a seed; 0 started with one more masked position so only compare
    # the rows where both were masked at step 0: identical seeds + inputs -> identical draws
    l2 = np.repeat(logits[:1], 2, axis=0)
    t2, s2 = np.repeat(tokens[:1], 2, axis=0), np.repeat(state[:1], 2, axis=0)
    r = unmask_step(l2, t2, s2, [4, 4], threshold=0.3, temperature=1.0, block_idx=0, step=0)
    np.testing.assert_array_equal(r["tokens"][0], r["tokens"][1])
    np.testing.assert_array_equal(r["state"][0], r["state"][1])
    r2 = unmask_step(l2, t2, s2, [4, 5], threshold=-1.0, temperature=1.0, block_idx=0, step=0)
    assert not np.array_equal(r2["tokens"][0], r2["tokens"][1])


def test_tiny_enumeration():
    # d <= 3, V <= 3: check against a direct enumeration of the rule on python floats
    for seed in range(20):
        g = np.random.default_rng(100 + seed)
        d, V = int(g.integers(1, 4)), int(g.integers(2, 4))
        logits = g.standard_normal((1, d, V))
        state = g.integers(0, 3, size=(1, d)).astype(np.uint8)
        tokens = g.integers(0, V, size=(1, d)).astype(np.int32)
        theta = float(g.uniform(0.2, 0.8))
        r = unmask_step(logits, tokens, state, [seed], theta, 0.0, 0, 0)
        exp_tok, exp_st = tokens.copy(), state.copy()
        cands = []
        for i in range(d):
            if state[0, i] != MASKED:
                continue
            e = [math.exp(x) for x in logits[0, i]]
            p = [x / sum(e) for x in e]
            best = max(range(V), key=lambda v: (p[v], -v))
            cands.append((i, best, p[best]))
        chosen = [c for c in cands if c[2] > theta]
        if not chosen and cands:
            chosen = [max(cands, key=lambda c: (c[2], -c[0]))]
        for i, t, _ in chosen:
            exp_tok[0, i], exp_st[0, i] = t, COMMITTED
        np.testing.assert_array_equal(r["tokens"], exp_tok)
        np.testing.assert_array_equal(r["state"], exp_st)


def test_gumbel_max_samples_softmax_of_scaled_logits():
    # chi-square goodness of fit: argmax(l + T g) ~ softmax(l / T), V = 8, 20000 independent rows
    V, T, n = 8, 0.8, 20000
    l = np.array([0.0, 0.5, -1.0, 1.2, 0.3, -0.4, 0.9, -2.0])
    p = np.exp(l / T) / np.exp(l / T).sum()
    counts = np.zeros(V)
    logits = np.tile(l, (1, 50, 1))
    tokens = np.zeros((1, 50), dtype=np.int32)
    state = np.zeros((1, 50), dtype=np.uint8)
    for s in range(n // 50):
        r = unmask_step(logits, tokens, state, [1000 + s], threshold=-1.0, temperature=T, block_idx=0, step=0)
        counts += np.bincount(r["tokens"][0], minlength=V)
    chi2 = float(((counts - n * p) ** 2 / (n * p)).sum())
    assert chi2 < 24.3                          # chi-square(7) 0.1 % critical value
    # confidence reported is the noise-free probability of the *chosen* token
    sm = np.exp(l) / np.exp(l).sum()
    np.testing.assert_allclose(r["conf"][0], sm[r["tokens"][0]], rtol=1e-13)


def test_planted_mistakes_are_caught():
    """The pins above must fail for plausible slips; spot-check three by planting them in copies
    of the oracle's arithmetic (on the CPU)."""
    l = np.array([0.0, 2.0, 1.0])
    conf_ok = math.exp(2.0) / (1 + math.exp(2.0) + math.exp(1.0))
    r = unmask_step(l[None, None], np.zeros((1, 1), np.int32), np.zeros((1, 1), np.uint8), [0], 0.0, 0.0, 0, 0)
    assert abs(r["conf"][0, 0] - conf_ok) < 1e-15
    wrong_no_max_term = math.exp(2.0) / (1 + math.exp(1.0))           # dropped term
    wrong_sign = math.exp(-2.0) / (1 + math.exp(-2.0) + math.exp(-1.0))
    assert abs(r["conf"][0, 0] - wrong_no_max_term) > 1e-2
    assert abs(r["conf"][0, 0] - wrong_sign) > 1e-2
