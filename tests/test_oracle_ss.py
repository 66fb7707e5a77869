"""Pins of the Scaffold Speculative Decoding oracle (Sec. 3.3): whatever the drafts are, the block
ends up with exactly the tokens plain left-to-right AR decoding would produce; scaffold tokens are
never touched; every draft / verify cycle commits at least one value position."""
import numpy as np

from oracle import MASKED, COMMITTED, SCAFFOLD
from oracle.ss import DRAFT, ss_accept, ss_draft

V = 23


def _ar_logits(prefix_tokens, position):
    """A toy AR head: the logits of `position` are a fixed pseudo-random function of the tokens
    before it (so a wrong earlier token changes every later prediction)."""
    h = 1469598103934665603
    for t in list(prefix_tokens) + [position]:
        h = ((h ^ (int(t) + 1)) * 1099511628211) & 0xFFFFFFFFFFFFFFFF
    return np.random.default_rng(h).standard_normal(V)


def _verify_logits(tokens_row):
    return np.stack([_ar_logits(tokens_row[:i], i) for i in range(len(tokens_row))])


def _ar_greedy(tokens_row, state_row):
    out = tokens_row.copy()
    for i in range(len(out)):
        if state_row[i] != SCAFFOLD:
            out[i] = int(np.argmax(_ar_logits(out[:i], i)))
    return out


def _run_ss(tokens, state, draft_quality, seed):
    """Draft / verify cycles until nothing is MASKED.  The drafts come from a "diffusion head" that
    agrees with the AR head with probability `draft_quality` per position."""
    g = np.random.default_rng(seed)
    tokens, state = tokens.copy(), state.copy()
    truth = np.stack([_ar_greedy(tokens[f], state[f]) for f in range(tokens.shape[0])])
    cycles = 0
    while np.any(state == MASKED):
        N, d = tokens.shape
        draft_logits = np.full((N, d, V), -5.0)
        for f in range(N):
            for i in range(d):
                guess = truth[f, i] if g.random() < draft_quality else int(g.integers(0, V))
                draft_logits[f, i, guess] = 5.0
        tokens, state = ss_draft(draft_logits, tokens, state, [1] * N, 0.0, 0, cycles)
        assert not np.any(state == MASKED)
        ar = np.stack([_verify_logits(tokens[f]) for f in range(N)])
        before = int(np.sum(state == COMMITTED))
        had_draft = np.any(state == DRAFT, axis=1)
        r = ss_accept(ar, tokens, state, [1] * N, 0.0, 0, cycles)
        tokens, state = r["tokens"], r["state"]
        assert not np.any(state == DRAFT)
        assert int(np.sum(state == COMMITTED)) - before == int(r["n_accepted"].sum())
        assert np.all(r["n_accepted"][had_draft] >= 1) and np.all(r["n_accepted"][~had_draft] == 0)
        cycles += 1
        assert cycles <= tokens.shape[1]
    return tokens, state, truth, cycles


def _block(N=3, d=12, scaffold=(0, 1, 5, 9)):
    tokens = np.full((N, d), V - 1, dtype=np.int32)
    state = np.full((N, d), MASKED, dtype=np.uint8)
    for i in scaffold:
        tokens[:, i] = 3 + i % 5
        state[:, i] = SCAFFOLD
    return tokens, state


def test_ss_output_equals_plain_ar_decoding_for_any_draft_quality():
    for quality, seed in ((1.0, 1), (0.7, 2), (0.3, 3), (0.0, 4)):
        tokens, state = _block()
        out, st, truth, cycles = _run_ss(tokens, state, quality, seed)
        np.testing.assert_array_equal(out, truth)
        assert np.all((st == COMMITTED) | (st == SCAFFOLD))
        np.testing.assert_array_equal(out[state == SCAFFOLD], tokens[state == SCAFFOLD])
        if quality == 1.0:
            assert cycles == 1                      # perfect drafts: one draft + one verify pass
        if quality == 0.0:
            assert cycles >= 2                      # the bonus token alone advances each cycle


def test_accept_scan_by_hand():
    # 6 positions: S D D D S D ; the verifier agrees on the first draft, disagrees on the second
    tokens = np.array([[7, 1, 2, 3, 8, 4]], dtype=np.int32)
    state = np.array([[SCAFFOLD, DRAFT, DRAFT, DRAFT, SCAFFOLD, DRAFT]], dtype=np.uint8)
    ar = np.zeros((1, 6, V))
    ar[0, 1, 1] = 1.0          # agrees
    ar[0, 2, 9] = 1.0          # disagrees: 9 replaces 2
    ar[0, 3, 3] = 1.0          # would agree, but comes after the rejection
    ar[0, 5, 4] = 1.0
    r = ss_accept(ar, tokens, state, [0], 0.0, 0, 0)
    assert r["tokens"].tolist() == [[7, 1, 9, 3, 8, 4]]
    assert r["state"].tolist() == [[SCAFFOLD, COMMITTED, COMMITTED, MASKED, SCAFFOLD, MASKED]]
    assert r["n_accepted"].tolist() == [2] and r["n_left"].tolist() == [2]
    # nothing under verification: a no-op
    r2 = ss_accept(ar, r["tokens"], np.where(r["state"] == MASKED, COMMITTED, r["state"]).astype(np.uint8), [0], 0.0, 0, 0)
    assert r2["n_accepted"].tolist() == [0] and r2["n_left"].tolist() == [0]


def test_sampled_verifier_uses_the_rollouts_noise():
    tokens, state = _block(N=2, d=8, scaffold=(0, 4))
    g = np.random.default_rng(9)
    logits = g.standard_normal((2, 8, V))
    logits[1] = logits[0]
    t1, s1 = ss_draft(logits, tokens, state, [5, 5], 1.5, 2, 0)
    np.testing.assert_array_equal(t1[0], t1[1])             # equal seeds: equal rollouts
    t2, _ = ss_draft(logits, tokens, state, [5, 6], 1.5, 2, 0)
    assert not np.array_equal(t2[0], t2[1])
    ar = g.standard_normal((2, 8, V))
    ar[1] = ar[0]
    r = ss_accept(ar, t1, s1, [5, 5], 1.5, 2, 1)
    np.testing.assert_array_equal(r["tokens"][0], r["tokens"][1])
    np.testing.assert_array_equal(r["state"][0], r["state"][1])
