"""The block loop of Section Diffusion (test infrastructure).

Sec. 3.3 ("Section Diffusion"): starting from the pre-filled scaffold, value
positions of a block are unmasked iteratively while attending to the cached
context; a finished block joins the cache.  One iteration here = attention for
every layer, then one unmasking step; the loop ends when no rollout has a
MASKED position left; then the block's K/V are appended to each rollout's
private suffix.

The model between attention and logits is not part of this repository, so the
caller supplies, per step, the projections q/k/v of the block and the logits.
"""
import numpy as np

from . import MASKED
from .attention import bf16_bits_to_f64, decode_block_attention
from .unmask import unmask_step


def _widen(x):
    x = np.asarray(x)
    return bf16_bits_to_f64(x) if x.dtype == np.uint16 else x.astype(np.float64)


def decode_block(forkset, inputs_for_step, tokens, state, threshold, temperature,
                 block_idx, scale, max_steps=None, want_attention=True):
    """Run the loop for one block.

    inputs_for_step(t) -> dict(q=[L][N,d,Hq,D], k=[L][N,d,Hkv,D], v=[L][...],
    logits=[N,d,V]) for denoising step t.  Returns dict(tokens, state, steps,
    committed_per_step=[steps][N], attn=[steps][L] outputs (if wanted)).
    """
    tokens = np.array(tokens, dtype=np.int32, copy=True)
    state = np.array(state, dtype=np.uint8, copy=True)
    n_layers = len(forkset.prefix_k)
    d = tokens.shape[1]
    if max_steps is None:
        max_steps = d
    committed, attn = [], []
    t = 0
    last = None
    while np.any(state == MASKED):
        assert t < max_steps, "a block must finish within block_size steps"
        last = inputs_for_step(t)
        if want_attention:
            outs = []
            for layer in range(n_layers):
                outs.append(decode_block_attention(
                    _widen(last["q"][layer]), _widen(last["k"][layer]), _widen(last["v"][layer]),
                    _widen(forkset.prefix_k[layer]), _widen(forkset.prefix_v[layer]),
                    [_widen(s) for s in forkset.suffix_k[layer]],
                    [_widen(s) for s in forkset.suffix_v[layer]], scale))
            attn.append(outs)
        r = unmask_step(_widen(last["logits"]), tokens, state, forkset.seeds,
                        threshold, temperature, block_idx, t)
        tokens, state = r["tokens"], r["state"]
        committed.append(r["n_committed"].copy())
        t += 1
    if last is not None:
        for layer in range(n_layers):
            forkset.kv_commit(layer, last["k"][layer], last["v"][layer])
    return dict(tokens=tokens, state=state, steps=t, committed_per_step=committed, attn=attn)
