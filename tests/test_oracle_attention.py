"""Pins for the attention oracle: special cases with library or closed-form
answers, brute force on tiny inputs, and invariants a wrong mask, index or
transposed operand would break."""
import math

import numpy as np
import torch

from oracle.attention import (bf16_bits_to_f64, block_causal_attention,
                              causal_block_attention_rows, decode_block_attention)


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


def _sdpa(q, k, v, mask=None, causal=False, scale=None):
    # torch CPU fp64 scaled-dot-product attention, [T,H,D] -> [T,H,D]
    tq, tk, tv = (torch.from_numpy(np.ascontiguousarray(x)).permute(1, 0, 2)[None] for x in (q, k, v))
    m = None if mask is None else torch.from_numpy(mask)[None, None]
    o = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=m, is_causal=causal, scale=scale)
    return o[0].permute(1, 0, 2).numpy()


def test_block_size_one_is_causal_attention():
    T, H, D = 13, 3, 8
    q, k, v = _rand((T, H, D), 1), _rand((T, H, D), 2), _rand((T, H, D), 3)
    o = block_causal_attention(q, k, v, np.arange(T), 0.37)
    np.testing.assert_allclose(o, _sdpa(q, k, v, causal=True, scale=0.37), rtol=1e-12, atol=1e-13)


def test_single_block_is_bidirectional_attention():
    T, H, D = 11, 2, 16
    q, k, v = _rand((T, H, D), 4), _rand((T, H, D), 5), _rand((T, H, D), 6)
    o = block_causal_attention(q, k, v, np.zeros(T, dtype=int), 0.25)
    np.testing.assert_allclose(o, _sdpa(q, k, v, scale=0.25), rtol=1e-12, atol=1e-13)


def test_brute_force_tiny():
    # every term written out with scalar math on T = 5, blocks (0,0,1,1,2)
    T, H, D = 5, 1, 2
    bid = [0, 0, 1, 1, 2]
    q, k, v = _rand((T, H, D), 7), _rand((T, H, D), 8), _rand((T, H, D), 9)
    o = block_causal_attention(q, k, v, np.array(bid), 1.0)
    visible = {0: [0, 1], 1: [0, 1], 2: [0, 1, 2, 3], 3: [0, 1, 2, 3], 4: [0, 1, 2, 3, 4]}
    for i in range(T):
        w = [math.exp(sum(q[i, 0, c] * k[j, 0, c] for c in range(D))) for j in visible[i]]
        z = sum(w)
        for c in range(D):
            ref = sum(wj / z * v[j, 0, c] for wj, j in zip(w, visible[i]))
            assert abs(o[i, 0, c] - ref) < 1e-12


def test_general_mask_matches_library_and_gqa_repeat():
    T, Hq, Hkv, D = 14, 4, 2, 8
    bid = np.array([0] * 5 + [1] * 3 + [2] * 4 + [3] * 2)
    q, k, v = _rand((T, Hq, D), 10), _rand((T, Hkv, D), 11), _rand((T, Hkv, D), 12)
    o = block_causal_attention(q, k, v, bid, 0.5)
    # GQA == MHA with each KV head repeated G times (h -> h // G)
    kr, vr = np.repeat(k, Hq // Hkv, axis=1), np.repeat(v, Hq // Hkv, axis=1)
    mask = bid[None, :] <= bid[:, None]
    np.testing.assert_allclose(o, _sdpa(q, kr, vr, mask=mask, scale=0.5), rtol=1e-12, atol=1e-13)
    # a later block never leaks: changing block 3's K/V leaves blocks 0-2 untouched
    k2, v2 = k.copy(), v.copy()
    k2[12:] += 5.0
    v2[12:] -= 3.0
    o2 = block_causal_attention(q, k2, v2, bid, 0.5)
    np.testing.assert_array_equal(o[:12], o2[:12])
    assert np.max(np.abs(o[12:] - o2[12:])) > 1e-3


def test_decode_form_equals_definition_form():
    N, d, Hq, Hkv, D, P = 3, 4, 4, 2, 8, 9
    S = [0, 4, 8]
    pk, pv = _rand((P, Hkv, D), 20), _rand((P, Hkv, D), 21)
    sk = [_rand((s, Hkv, D), 30 + f) for f, s in enumerate(S)]
    sv = [_rand((s, Hkv, D), 40 + f) for f, s in enumerate(S)]
    q = _rand((N, d, Hq, D), 22)
    kb, vb = _rand((N, d, Hkv, D), 23), _rand((N, d, Hkv, D), 24)
    o = decode_block_attention(q, kb, vb, pk, pv, sk, sv, 0.3)
    for f in range(N):
        T = P + S[f] + d
        k_all = np.concatenate([pk, sk[f], kb[f]])
        v_all = np.concatenate([pv, sv[f], vb[f]])
        q_all = np.concatenate([_rand((P + S[f], Hq, D), 50 + f), q[f]])
        nb_suffix = S[f] // d
        bid = np.array([0] * P + [1 + j for j in range(nb_suffix) for _ in range(d)] + [1 + nb_suffix] * d)
        assert len(bid) == T
        full = block_causal_attention(q_all, k_all, v_all, bid, 0.3)
        np.testing.assert_allclose(o[f], full[-d:], rtol=1e-12, atol=1e-13)


def test_key_permutation_invariance_and_closed_forms():
    N, d, Hq, Hkv, D, P = 1, 3, 2, 1, 4, 7
    pk, pv = _rand((P, Hkv, D), 60), _rand((P, Hkv, D), 61)
    kb, vb = _rand((N, d, Hkv, D), 62), _rand((N, d, Hkv, D), 63)
    q = _rand((N, d, Hq, D), 64)
    empty = [np.zeros((0, Hkv, D))]
    o = decode_block_attention(q, kb, vb, pk, pv, empty, empty, 0.7)
    perm = np.random.default_rng(65).permutation(P)
    o_perm = decode_block_attention(q, kb, vb, pk[perm], pv[perm], empty, empty, 0.7)
    np.testing.assert_allclose(o, o_perm, rtol=1e-12, atol=1e-14)
    # permuting the block's own keys (with their values) changes nothing either:
    # inside a block attention is bidirectional, so key order is irrelevant
    bp = np.array([2, 0, 1])
    o_bperm = decode_block_attention(q, kb[:, bp], vb[:, bp], pk, pv, empty, empty, 0.7)
    np.testing.assert_allclose(o, o_bperm, rtol=1e-12, atol=1e-14)
    # q = 0 -> uniform weights -> mean of every visible value row
    o0 = decode_block_attention(np.zeros_like(q), kb, vb, pk, pv, empty, empty, 0.7)
    mean_v = np.concatenate([pv, vb[0]]).mean(axis=0)
    for i in range(d):
        for h in range(Hq):
            np.testing.assert_allclose(o0[0, i, h], mean_v[0], rtol=1e-13)
    # one dominating key -> that key's value row
    kdom = pk.copy()
    kdom[3, 0] = 1e4 * q[0, 1, 0] / np.dot(q[0, 1, 0], q[0, 1, 0])
    od = decode_block_attention(q, kb, vb, kdom, pv, empty, empty, 1.0)
    np.testing.assert_allclose(od[0, 1, 0], pv[3, 0], rtol=1e-9, atol=1e-12)
    # shifting every score of a row by a constant (k -> k + c*q/|q|^2 changes all scores of that
    # query by c) leaves that query's output unchanged
    shift = 3.0 * q[0, 2, 1] / np.dot(q[0, 2, 1], q[0, 2, 1]) / 0.7
    os_ = decode_block_attention(q, kb + shift, vb, pk + shift, pv, empty, empty, 0.7)
    np.testing.assert_allclose(os_[0, 2, 1], o[0, 2, 1], rtol=1e-10, atol=1e-12)


def test_forks_share_prefix_but_not_suffix():
    N, d, Hq, Hkv, D, P = 2, 2, 2, 1, 4, 5
    pk, pv = _rand((P, Hkv, D), 70), _rand((P, Hkv, D), 71)
    q1 = _rand((1, d, Hq, D), 72)
    kb1, vb1 = _rand((1, d, Hkv, D), 73), _rand((1, d, Hkv, D), 74)
    q, kb, vb = np.repeat(q1, N, 0), np.repeat(kb1, N, 0), np.repeat(vb1, N, 0)
    s0k, s0v = _rand((2, Hkv, D), 75), _rand((2, Hkv, D), 76)
    same = decode_block_attention(q, kb, vb, pk, pv, [s0k, s0k], [s0v, s0v], 0.5)
    np.testing.assert_array_equal(same[0], same[1])
    diff = decode_block_attention(q, kb, vb, pk, pv, [s0k, s0k + 1.0], [s0v, s0v], 0.5)
    np.testing.assert_array_equal(diff[0], same[0])          # fork 0 unaffected by fork 1's suffix
    assert np.max(np.abs(diff[1] - same[1])) > 1e-6
    # N-fork batched call == N single-fork calls
    for f in range(N):
        one = decode_block_attention(q[f:f + 1], kb[f:f + 1], vb[f:f + 1], pk, pv,
                                     [[s0k, s0k + 1.0][f]], [s0v], 0.5)
        np.testing.assert_array_equal(one[0], diff[f])


def test_causal_rows_form_is_block_size_one():
    N, d, Hq, Hkv, D, P = 2, 5, 2, 1, 4, 6
    pk, pv = _rand((P, Hkv, D), 80), _rand((P, Hkv, D), 81)
    q = _rand((N, d, Hq, D), 82)
    kb, vb = _rand((N, d, Hkv, D), 83), _rand((N, d, Hkv, D), 84)
    sk = [_rand((3, Hkv, D), 85), _rand((0, Hkv, D), 86)]
    sv = [_rand((3, Hkv, D), 87), _rand((0, Hkv, D), 88)]
    o = causal_block_attention_rows(q, kb, vb, pk, pv, sk, sv, 0.4)
    for f in range(N):
        k_all = np.concatenate([pk, sk[f], kb[f]])
        v_all = np.concatenate([pv, sv[f], vb[f]])
        T = len(k_all)
        q_all = np.concatenate([np.zeros((T - d, Hq, D)), q[f]])
        bid = np.array([0] * (T - d) + list(range(1, d + 1)))
        full = block_causal_attention(q_all, k_all, v_all, bid, 0.4)
        np.testing.assert_allclose(o[f], full[-d:], rtol=1e-12, atol=1e-13)


def test_bf16_widening_is_exact():
    bits = np.array([0x3F80, 0xBF80, 0x0000, 0x4049, 0x7F7F, 0x0080], dtype=np.uint16)
    ref = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).double().numpy()
    np.testing.assert_array_equal(bf16_bits_to_f64(bits), ref)
