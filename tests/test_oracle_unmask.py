"""Pins for the Philox/Gumbel generator and the unmasking rule of the oracle."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import MASKED, COMMITTED, SCAFFOLD
from oracle.philox import (exponential_row, exponential_scalar, fine_bits, group_words, gumbel_row,
                           leader_exponential, philox4x32_scalar, philox4x32_vec)
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


def test_leader_map_is_open_interval_and_monotone():
    # U = (h + (f + 0.5) 2^-23) / 2^28 tiles (0, 1) in steps of 2^-51; E = -ln(U) / 16 falls as U grows
    top = 2 ** 28 - 1
    words = np.array([0, 0, 0, 1, top // 2, top, top], dtype=np.uint64) << np.uint64(4)
    f = np.array([0, 1, 2 ** 23 - 1, 0, 5, 0, 2 ** 23 - 1])
    e = leader_exponential(words, f)
    assert np.all(np.diff(e) < 0) and np.all(e > 0) and np.all(np.isfinite(e))
    assert e[0] == -math.log(2.0 ** -52) / 16                      # smallest U = 2^-52
    assert abs(e[-1] - 2.0 ** -52 / 16) < 1e-30                    # largest U = 1 - 2^-52: E = 2^-52 / 16 + O(2^-104)
    # the low four bits of the word (the leader's place) do not enter
    assert np.array_equal(leader_exponential(words + np.uint64(9), f), e)
    g = -np.log(e)
    assert -1.0 < g[0] and g[-1] < 38.9


def test_gumbel_row_layout_and_independence_from_vocab_size():
    seed = 0xDEADBEEFCAFEF00D
    V = 16 * 1024 + 40
    a = gumbel_row(seed, 3, 2, 5, V)
    b = gumbel_row(seed, 3, 2, 5, V + 23)
    np.testing.assert_array_equal(a, b[:V])
    np.testing.assert_array_equal(gumbel_row(seed, 3, 2, 5, 37), a[:37])    # a cut group included
    key = (seed & 0xFFFFFFFF, seed >> 32)
    words = group_words(seed, 3, 2, 5, V)
    fb = fine_bits(seed, 3, 2, 5, V + 16)
    # group j: word j % 4 of counter (j // 4, pos, step, block); fine: top 23 bits of word v % 4 of
    # counter (v // 4, pos + 2^31, step, block); both under key (lo, hi).  Spelled out here once more
    # on Python integers, and compared with the one-id-at-a-time definition of the oracle.
    seen_leader = seen_other = 0
    for v in (0, 5, 18, 63, 64, 255 * 16 + 3, 256 * 16 + 1, 700 * 16 + 15, 1023 * 16, 1024 * 16 + 7, V - 1) + tuple(range(32, 64)):
        j = v // 16
        R = philox4x32_scalar((j // 4, 5, 2, 3), key)[j % 4]
        assert int(words[j]) == R
        lead = 16 * j + R % 16
        f_lead = philox4x32_scalar((lead // 4, 5 + 2 ** 31, 2, 3), key)[lead % 4] >> 9
        assert int(fb[lead]) == f_lead
        U = ((R >> 4) + (f_lead + 0.5) * 2.0 ** -23) * 2.0 ** -28
        e = -math.log(U) / 16
        if v != lead:
            f_v = philox4x32_scalar((v // 4, 5 + 2 ** 31, 2, 3), key)[v % 4] >> 9
            e += -math.log((f_v + 0.5) * 2.0 ** -23)
            seen_other += 1
        else:
            seen_leader += 1
        assert abs(a[v] + math.log(e)) <= 1e-12 * max(1.0, abs(a[v]))
        assert e == exponential_scalar(seed, 3, 2, 5, v)
    assert seen_leader >= 2 and seen_other >= 20
    # every counter field and the seed matter
    for other in (gumbel_row(seed + 1, 3, 2, 5, 37), gumbel_row(seed, 4, 2, 5, 37),
                  gumbel_row(seed, 3, 1, 5, 37), gumbel_row(seed, 3, 2, 6, 37),
                  gumbel_row(seed ^ (1 << 40), 3, 2, 5, 37)):
        assert not np.array_equal(a[:37], other)


def test_row_function_equals_the_scalar_definition_everywhere():
    # the vectorised row against the one-id-at-a-time definition on every id of a short row and on
    # random ids of a long one (both rows cut their last group)
    for seed, blk, step, pos, V, ids in ((7, 0, 0, 0, 100, range(100)),
                                         (2 ** 63 + 11, 5, 9, 127, 151936 - 3,
                                          np.random.default_rng(3).integers(0, 151936 - 3, 300))):
        e = exponential_row(seed, blk, step, pos, V)
        for v in ids:
            ref = exponential_scalar(seed, blk, step, pos, int(v))
            assert abs(e[v] - ref) <= 1e-13 * ref


def test_words_are_the_stream_in_order_and_streams_do_not_overlap():
    # the group words are the Philox blocks 0, 1, 2, ... of (position, step, block) read word by
    # word; the fine bits come from the blocks of (position + 2^31, step, block): no counter is
    # used by both, whatever the position (positions stay far below 2^31)
    seed, key = 99, (99, 0)
    words = group_words(seed, 1, 2, 3, 16 * 12)
    flat = [x for c in range(3) for x in philox4x32_scalar((c, 3, 2, 1), key)]
    assert [int(x) for x in words] == flat
    fb = fine_bits(seed, 1, 2, 3, 12)
    flat_f = [x >> 9 for c in range(3) for x in philox4x32_scalar((c, 3 + 2 ** 31, 2, 1), key)]
    assert [int(x) for x in fb] == flat_f


def test_group_word_bounds_every_draw_of_the_group():
    # what lets an implementation skip the per-id stream: the word of a group alone bounds the 16
    # draws of the group, E[v] >= -ln((h + 1) / 2^28) / 16 with h = word >> 4; a word below 0xFF000000
    # (255 of 256 groups) caps them at g < 8.3158, one below 0xFC000000 (63 of 64) at g < 6.9237
    V = 50000
    e = exponential_row(777, 1, 4, 9, V)
    words = group_words(777, 1, 4, 9, V)
    h = (words >> np.uint64(4)).astype(np.float64)
    floor = np.repeat(-np.log((h + 1.0) * 2.0 ** -28) / 16, 16)[:V]
    ceil_leader = np.repeat(-np.log(np.maximum(h, 0.5) * 2.0 ** -28) / 16, 16)[:V]
    assert np.all(e >= floor)
    grp_min = np.minimum.reduceat(e, np.arange(0, V, 16))
    lead = np.arange(len(words)) * 16 + (words & np.uint64(15)).astype(np.int64)
    inside = lead < V
    np.testing.assert_array_equal(grp_min[inside], e[lead[inside]])           # the leader holds the minimum
    assert np.all(e[lead[inside]] <= ceil_leader[lead[inside]])
    g = -np.log(e)
    for top_word, cap, share in ((0xFF000000, 8.3158, 256), (0xFC000000, 6.9237, 64)):
        plain = np.repeat(words < np.uint64(top_word), 16)[:V]
        assert np.all(g[plain] < cap)
        assert 0.6 / share < 1.0 - plain.mean() < 1.6 / share
    # the leader's place is uniform over the 16 ids and unrelated to the minimum
    places = (words & np.uint64(15)).astype(int)
    counts = np.bincount(places, minlength=16)
    chi2 = float(((counts - len(places) / 16) ** 2 / (len(places) / 16)).sum())
    assert chi2 < 37.7                                   # chi-square(15) 0.1 % critical value
    assert abs(np.corrcoef(places, h)[0, 1]) < 0.05


def test_gumbel_uniformity_ks():
    # Kolmogorov-Smirnov distance of exp(-exp(-g)) = u from U(0,1) on 2e5 draws
    g = gumbel_row(12345, 0, 0, 0, 200000)
    u = np.sort(np.exp(-np.exp(-g)))
    n = len(u)
    dist = np.max(np.abs(u - (np.arange(n) + 0.5) / n))
    assert dist < 1.63 / math.sqrt(n)          # 1 % critical value


def test_draws_inside_a_group_are_independent_exponentials():
    # the race construction must not show: group minima are Exp(1) / 16, neighbours inside a group are
    # uncorrelated, and so are a group's minimum and the excess of its other ids
    V = 320000
    e = exponential_row(4242, 2, 1, 3, V).reshape(-1, 16)
    m = np.sort(e.min(axis=1) * 16)
    n = len(m)
    cdf = 1.0 - np.exp(-m)
    assert np.max(np.abs(cdf - (np.arange(n) + 0.5) / n)) < 1.63 / math.sqrt(n)
    u = np.exp(-e)
    for a_, b_ in ((0, 1), (3, 12), (7, 8), (14, 15)):
        assert abs(np.corrcoef(u[:, a_], u[:, b_])[0, 1]) < 0.02
    second = np.sort(e, axis=1)[:, 1] - e.min(axis=1)              # gap to the runner-up: Exp(1) / 15
    s2 = np.sort(second * 15)
    assert np.max(np.abs(1.0 - np.exp(-s2) - (np.arange(n) + 0.5) / n)) < 1.63 / math.sqrt(n)
    assert abs(np.corrcoef(e.min(axis=1), second)[0, 1]) < 0.02
    # every id alone is Exp(1), leader or not: mean 1, variance 1 per column
    assert np.all(np.abs(e.mean(axis=0) - 1.0) < 0.03) and np.all(np.abs(e.var(axis=0) - 1.0) < 0.08)


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


def _winner_counts(l, T, n, seed0):
    """argmax(l + T g) over n independent rows (positions x seeds) through unmask_step."""
    V = len(l)
    rows = 50
    logits = np.tile(np.asarray(l, dtype=np.float64), (1, rows, 1))
    tokens = np.zeros((1, rows), dtype=np.int32)
    state = np.zeros((1, rows), dtype=np.uint8)
    counts = np.zeros(V)
    lead_wins = 0
    for s in range(n // rows):
        r = unmask_step(logits, tokens, state, [seed0 + s], threshold=-1.0, temperature=T, block_idx=2, step=s % 7)
        counts += np.bincount(r["tokens"][0], minlength=V)
        for i in range(rows):
            w = group_words(seed0 + s, 2, s % 7, i, V)
            t = int(r["tokens"][0, i])
            lead_wins += int(16 * (t // 16) + int(w[t // 16]) % 16 == t)
    return counts, lead_wins


def test_gumbel_max_over_several_groups_leaders_and_followers_win():
    # V = 48: three groups of 16.  The race construction gives every group one id (its leader) a
    # head start; the frequencies must still be softmax(l / T), whether the winner is a leader or
    # not.  chi-square(47): 0.1 % critical value 82.7
    V, T, n = 48, 0.7, 20000
    g = np.random.default_rng(11)
    l = g.standard_normal(V) * 1.2
    p = np.exp(l / T) / np.exp(l / T).sum()
    counts, lead_wins = _winner_counts(l, T, n, 5000)
    chi2 = float(((counts - n * p) ** 2 / (n * p)).sum())
    assert chi2 < 82.7
    # P(winner is its group's leader) = sum_v p_v P(v leads | v wins); a leader is the smallest of 16
    # draws, so it wins far more often than 1 / 16 of the time, yet not always
    assert 0.25 * n < lead_wins < 0.95 * n
    # per group: the group's total mass
    grp = counts.reshape(3, 16).sum(axis=1)
    pg = p.reshape(3, 16).sum(axis=1)
    assert float(((grp - n * pg) ** 2 / (n * pg)).sum()) < 13.8       # chi-square(2) 0.1 %


def test_equal_logits_give_a_uniform_winner():
    # all logits equal: the noise alone decides, every id of every group equally often
    V, n = 48, 14400
    counts, lead_wins = _winner_counts(np.full(V, 1.5), 1.0, n, 9000)
    chi2 = float(((counts - n / V) ** 2 / (n / V)).sum())
    assert chi2 < 82.7
    assert lead_wins == n          # with equal logits the winner is the id with the smallest E: a leader


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
