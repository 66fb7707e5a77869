"""Pins for the fork/commit cache, trajectory averaging, the block loop and the
synthetic input recipes."""
import numpy as np

from oracle import MASKED, COMMITTED, SCAFFOLD
from oracle.attention import bf16_bits_to_f64, decode_block_attention
from oracle.average import average_rollouts
from oracle.cache import ForkSet
from oracle.decode import decode_block
from paper_2605_23163_b200 import synth


def test_average_closed_forms():
    g = np.random.default_rng(0)
    t = g.standard_normal((5, 10, 2)).astype(np.float32)
    out = average_rollouts(t)
    np.testing.assert_allclose(out, t.astype(np.float64).mean(axis=0), rtol=1e-15, atol=1e-16)
    np.testing.assert_array_equal(average_rollouts(t[:1]), t[0].astype(np.float64))       # N = 1 identity
    np.testing.assert_allclose(average_rollouts(t[g.permutation(5)]), out, rtol=1e-14, atol=1e-15)
    # arithmetic sequence: mean of k * base over k = 1..N is base * (N + 1) / 2
    base = g.standard_normal((10, 2))
    seq = np.stack([k * base for k in range(1, 8)])
    np.testing.assert_allclose(average_rollouts(seq), base * 4.0, rtol=1e-14)


def test_fork_commit_is_private_and_bit_exact():
    g = np.random.default_rng(1)
    pk = [g.integers(0, 2 ** 16, size=(6, 2, 4)).astype(np.uint16)]
    pv = [g.integers(0, 2 ** 16, size=(6, 2, 4)).astype(np.uint16)]
    fs = ForkSet(pk, pv, 3, [1, 2, 3])
    pk_before = pk[0].copy()
    kb = g.integers(0, 2 ** 16, size=(3, 5, 2, 4)).astype(np.uint16)
    vb = g.integers(0, 2 ** 16, size=(3, 5, 2, 4)).astype(np.uint16)
    fs.kv_commit(0, kb, vb)
    kb2 = g.integers(0, 2 ** 16, size=(3, 5, 2, 4)).astype(np.uint16)
    fs.kv_commit(0, kb2, vb)
    for f in range(3):
        assert fs.suffix_len(f) == 10
        np.testing.assert_array_equal(fs.suffix_k[0][f][:5], kb[f])
        np.testing.assert_array_equal(fs.suffix_k[0][f][5:], kb2[f])
        np.testing.assert_array_equal(fs.suffix_v[0][f][5:], vb[f])
    np.testing.assert_array_equal(fs.prefix_k[0], pk_before)       # the prefix is never written
    assert fs.prefix_k[0] is pk[0]                                  # shared, not copied


def test_attention_after_commit_equals_block_passed_as_suffix():
    w = synth.small_variant(synth.workload("tts"), prefix_len=40, vocab=64, n_forks=2, n_blocks=2)
    pk, pv = synth.make_prefix(w, 0)
    fs = ForkSet([pk], [pv], 2, synth.fork_seeds(w, 0))
    q0, k0, v0 = synth.make_qkv(w, 0, 0, 0, 0)
    q1, k1, v1 = synth.make_qkv(w, 0, 0, 1, 0)
    fs.kv_commit(0, k0, v0)
    W = bf16_bits_to_f64
    a = decode_block_attention(W(q1), W(k1), W(v1), W(pk), W(pv),
                               [W(s) for s in fs.suffix_k[0]], [W(s) for s in fs.suffix_v[0]], 0.1)
    b = decode_block_attention(W(q1), W(k1), W(v1), W(pk), W(pv),
                               [W(k0[f]) for f in range(2)], [W(v0[f]) for f in range(2)], 0.1)
    np.testing.assert_array_equal(a, b)


def test_fork_after_deterministic_blocks_equals_fork_from_a_longer_prefix():
    # Sec. 3.4: decode the deterministic sections once (one rollout), then fork.  Forking after k
    # blocks were appended to the prefix is the same thing, bit for bit, as forking from a prefix
    # that contained them from the start; the rollouts' attention then equals attention over the
    # short prefix with those blocks handed to every rollout as its suffix.
    w = synth.small_variant(synth.workload("tts"), prefix_len=24, vocab=64, n_forks=3, n_blocks=4)
    pk, pv = synth.make_prefix(w, 0)
    one = ForkSet([pk], [pv], 1, [7])
    blocks = []
    for b in range(2):
        _, kb, vb = synth.make_qkv(w, 0, 0, b, 0)
        blocks.append((kb[:1], vb[:1]))
        one.extend_prefix(0, kb[:1], vb[:1])
    assert one.prefix_k[0].shape[0] == 24 + 2 * w.scenes[0].block_len
    np.testing.assert_array_equal(one.prefix_k[0][:24], pk)                 # the old part is untouched
    np.testing.assert_array_equal(one.prefix_k[0][24:24 + 32], blocks[0][0][0])
    np.testing.assert_array_equal(one.prefix_v[0][24 + 32:], blocks[1][1][0])
    assert pk.shape[0] == 24                                                 # the caller's array was not grown in place
    forked = one.fork(3, [1, 2, 3])
    long_k = np.concatenate([pk, blocks[0][0][0], blocks[1][0][0]], axis=0)
    long_v = np.concatenate([pv, blocks[0][1][0], blocks[1][1][0]], axis=0)
    direct = ForkSet([long_k], [long_v], 3, [1, 2, 3])
    np.testing.assert_array_equal(forked.prefix_k[0], direct.prefix_k[0])
    np.testing.assert_array_equal(forked.prefix_v[0], direct.prefix_v[0])
    assert all(forked.suffix_len(f) == 0 for f in range(3)) and forked.seeds == [1, 2, 3]
    q, k, v = synth.make_qkv(w, 0, 0, 2, 0)
    W = bf16_bits_to_f64
    none = [np.zeros((0, w.n_kv_heads, w.head_dim))] * 3
    a = decode_block_attention(W(q), W(k), W(v), W(forked.prefix_k[0]), W(forked.prefix_v[0]), none, none, 0.1)
    as_suffix_k = [W(np.concatenate([blocks[0][0][0], blocks[1][0][0]], axis=0))] * 3
    as_suffix_v = [W(np.concatenate([blocks[0][1][0], blocks[1][1][0]], axis=0))] * 3
    b_ = decode_block_attention(W(q), W(k), W(v), W(pk), W(pv), as_suffix_k, as_suffix_v, 0.1)
    np.testing.assert_array_equal(a, b_)
    # a set with several rollouts, or one that has a private suffix, cannot extend the prefix
    import pytest
    with pytest.raises(AssertionError):
        forked.extend_prefix(0, k[:1], v[:1])
    one.kv_commit(0, k[:1], v[:1])
    with pytest.raises(AssertionError):
        one.extend_prefix(0, k[:1], v[:1])


def _run_block(w, block=0, identical_seeds=False, temperature=None):
    pk, pv = synth.make_prefix(w, 0)
    fs = ForkSet([pk], [pv], w.scenes[0].n_forks, synth.fork_seeds(w, 0, identical=identical_seeds))
    tokens, state = synth.make_block_template(w, 0, block)

    def inputs(t):
        q, k, v = synth.make_qkv(w, 0, 0, block, t)
        lg = synth.make_logits(w, 0, block, t)
        if identical_seeds:      # identical inputs for every rollout
            q, k, v, lg = (np.repeat(x[:1], x.shape[0], axis=0) for x in (q, k, v, lg))
        if w.logits_dtype == "bf16":
            lg = bf16_bits_to_f64(lg)
        return dict(q=[q], k=[k], v=[v], logits=lg)

    r = decode_block(fs, inputs, tokens, state, w.threshold,
                     w.temperature if temperature is None else temperature, block,
                     1.0 / np.sqrt(w.head_dim), want_attention=False)
    return fs, tokens, state, r


def test_block_loop_tiny_workload_uses_fallback_every_step():
    w = synth.workload("tiny")
    fs, tokens, state, r = _run_block(w)
    sc = w.scenes[0]
    n_value = sc.block_len - sc.n_scaffold
    assert r["steps"] == n_value                       # never confident -> one commit per step
    assert all(int(c[0]) == 1 for c in r["committed_per_step"])
    frozen = state == SCAFFOLD
    np.testing.assert_array_equal(r["tokens"][frozen], tokens[frozen])
    assert np.all(r["state"][frozen] == SCAFFOLD) and np.all(r["state"][~frozen] == COMMITTED)
    assert fs.suffix_len(0) == sc.block_len


def test_block_loop_peaked_workload_and_identical_seeds():
    w = synth.small_variant(synth.workload("tts"), prefix_len=32, vocab=512, n_forks=3, n_blocks=1)
    fs, tokens, state, r = _run_block(w, identical_seeds=True)
    sc = w.scenes[0]
    assert 1 <= r["steps"] <= sc.block_len - sc.n_scaffold
    assert sum(int(c.sum()) for c in r["committed_per_step"]) == 3 * (sc.block_len - sc.n_scaffold)
    for f in (1, 2):                                   # same seed + same inputs -> same rollout
        np.testing.assert_array_equal(r["tokens"][f], r["tokens"][0])
    fs2, _, _, r2 = _run_block(w, identical_seeds=False)
    assert any(not np.array_equal(r2["tokens"][f], r2["tokens"][0]) for f in (1, 2))
    # every step commits at least one token in every unfinished rollout
    for c in r2["committed_per_step"][:-1]:
        assert np.all(c >= 0)
    assert all(c.sum() >= 1 for c in r2["committed_per_step"])


def test_synth_recipes():
    w = synth.workload("long_prefix")
    assert (w.group, w.scenes[0].block_len - w.scenes[0].n_scaffold) == (4, 38)
    row = synth.make_logits_row(w, 0, 0, 0, 3, 5)
    assert row.dtype == np.uint16 and row.shape == (w.vocab,)
    l = bf16_bits_to_f64(row)
    p = np.exp(l - l.max())
    p /= p.sum()
    assert 0.45 < p.max() < 0.999                      # sigmoid(U(0,6)) up to bf16 rounding of the peak
    np.testing.assert_array_equal(row, synth.make_logits_row(w, 0, 0, 0, 3, 5))      # reproducible
    assert not np.array_equal(row, synth.make_logits_row(w, 0, 0, 1, 3, 5))
    # bf16 rounding: nearest even, exact on representable values
    import torch
    x = np.random.default_rng(3).standard_normal(1000).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(synth.f32_to_bf16_bits(x), ref)
    sm = synth.workload("serving_mix")
    assert len(sm.scenes) == 16 and all(2048 <= s.prefix_len <= 12288 for s in sm.scenes)
    assert {s.n_forks for s in sm.scenes} <= {1, 4, 16} and {s.block_len for s in sm.scenes} <= {16, 32, 64}
    tok, st = synth.make_block_template(w, 0, 0)
    assert tok.shape == (32, 64) and (st[0] == SCAFFOLD).sum() == 26 and (st[0] == MASKED).sum() == 38
    tr = synth.tokens_to_trajectory(w, np.full((2, 200), 13, dtype=np.int32), np.zeros((2, 200), np.uint8))
    assert tr.shape == (2, 10, 2) and np.allclose(tr, -333.33)
