"""Block-causal attention in fp64 (test infrastructure, CPU oracle).

Sec. 3.1 ("Block-Causal Diffusion"): the output is split into blocks; a token
attends bidirectionally to every token of its own block and causally to the
prompt and to every earlier block, never to a later block.  With a block id
b(.) that does not decrease along the sequence (prompt = block 0) the visible
set of query i is { j : b(j) <= b(i) }.

Two forms are written out.  `block_causal_attention` is that definition on a
whole sequence.  `decode_block_attention` is what one denoising step needs:
the queries of the current block against the concatenation of a shared prefix
cache, the rollout's private suffix cache and the block's own keys (Sec. 3.3
"Section Diffusion": earlier sections come from the cache without
recomputation; Sec. 3.4: rollouts share the prefix cache).  The tests check
that the two agree.

Readings where the paper is silent: soft-max scale is an argument (1/sqrt(D)
by convention); grouped-query attention maps query head h to KV head
h // (Hq // Hkv); q and k arrive already position-encoded.
"""
import numpy as np


def bf16_bits_to_f64(bits):
    """Widen bfloat16 bit patterns (uint16) to float64 exactly."""
    bits = np.asarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def _softmax_rows(s):
    m = np.max(s, axis=-1, keepdims=True)
    e = np.exp(s - m)
    return e / np.sum(e, axis=-1, keepdims=True)


def block_causal_attention(q, k, v, block_id, scale):
    """Definition form.

    q: [T, Hq, D], k, v: [T, Hkv, D] (float64), block_id: [T] non-decreasing
    ints.  Returns o: [T, Hq, D] with
    o[i, h] = sum_{j : b(j) <= b(i)} softmax_j(scale * q[i, h] . k[j, h // G]) v[j, h // G].
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    block_id = np.asarray(block_id)
    T, Hq, D = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    assert Hq == G * Hkv and np.all(np.diff(block_id) >= 0)
    o = np.zeros_like(q)
    for i in range(T):
        vis = np.nonzero(block_id <= block_id[i])[0]
        for h in range(Hq):
            s = scale * (k[vis, h // G, :] @ q[i, h, :])
            p = _softmax_rows(s[None, :])[0]
            o[i, h, :] = p @ v[vis, h // G, :]
    return o


def decode_block_attention(q, k_blk, v_blk, prefix_k, prefix_v, suffix_k, suffix_v, scale):
    """Decode form for N rollouts forked from one prefix.

    q: [N, d, Hq, D]; k_blk, v_blk: [N, d, Hkv, D] (the current block);
    prefix_k, prefix_v: [P, Hkv, D], shared by every rollout;
    suffix_k, suffix_v: list of N arrays [S_f, Hkv, D], private per rollout.
    Every query of rollout f sees prefix + suffix_f + all d block keys of f.
    Returns o: [N, d, Hq, D] float64.
    """
    q = np.asarray(q, dtype=np.float64)
    N, d, Hq, D = q.shape
    Hkv = np.asarray(prefix_k).shape[1]
    G = Hq // Hkv
    assert Hq == G * Hkv
    o = np.zeros((N, d, Hq, D), dtype=np.float64)
    for f in range(N):
        keys = np.concatenate([np.asarray(prefix_k, dtype=np.float64),
                               np.asarray(suffix_k[f], dtype=np.float64).reshape(-1, Hkv, D),
                               np.asarray(k_blk[f], dtype=np.float64)], axis=0)
        vals = np.concatenate([np.asarray(prefix_v, dtype=np.float64),
                               np.asarray(suffix_v[f], dtype=np.float64).reshape(-1, Hkv, D),
                               np.asarray(v_blk[f], dtype=np.float64)], axis=0)
        for h in range(Hq):
            s = scale * (q[f, :, h, :] @ keys[:, h // G, :].T)      # [d, T]
            p = _softmax_rows(s)
            o[f, :, h, :] = p @ vals[:, h // G, :]
    return o


def causal_block_attention_rows(q, k_blk, v_blk, prefix_k, prefix_v, suffix_k, suffix_v, scale):
    """Block-size-1 mask inside the current block (the verifier pass of Scaffold
    Speculative Decoding, Sec. 3.3 step 3): query i of the block sees the cache
    and block keys 0..i only.  Same shapes as `decode_block_attention`."""
    q = np.asarray(q, dtype=np.float64)
    N, d, Hq, D = q.shape
    Hkv = np.asarray(prefix_k).shape[1]
    G = Hq // Hkv
    o = np.zeros((N, d, Hq, D), dtype=np.float64)
    for f in range(N):
        ctx_k = np.concatenate([np.asarray(prefix_k, dtype=np.float64),
                                np.asarray(suffix_k[f], dtype=np.float64).reshape(-1, Hkv, D)], axis=0)
        ctx_v = np.concatenate([np.asarray(prefix_v, dtype=np.float64),
                                np.asarray(suffix_v[f], dtype=np.float64).reshape(-1, Hkv, D)], axis=0)
        for i in range(d):
            keys = np.concatenate([ctx_k, np.asarray(k_blk[f, :i + 1], dtype=np.float64)], axis=0)
            vals = np.concatenate([ctx_v, np.asarray(v_blk[f, :i + 1], dtype=np.float64)], axis=0)
            for h in range(Hq):
                s = scale * (keys[:, h // G, :] @ q[f, i, h, :])
                p = _softmax_rows(s[None, :])[0]
                o[f, i, h, :] = p @ vals[:, h // G, :]
    return o
