"""Scaffold Speculative Decoding: the draft and the accept scan (test infrastructure, CPU oracle).

Sec. 3.3 ("Scaffold Speculative Decoding", Algorithm steps 1-3): per block, scaffold positions are
accepted as they are; one bidirectional pass of the diffusion head fills every masked value
position with a draft token; one causal pass of the AR head gives, for every position, the
distribution of that position given everything before it.  Going over the value positions from
left to right, a draft token is accepted while it equals the AR head's token; at the first
mismatch the AR head's token replaces the draft (the "bonus" token, always accepted) and every
later draft token of the block is discarded.  Sec. 3.4 puts the stochasticity of the trajectory
section inside this verifier: its token is a sample, not the arg-max.

Readings where the paper is silent: a discarded position goes back to MASKED and is drafted again
by the next draft / verify cycle of the block; the verifier's sample at temperature T is
argmax(logit + T * g) with the Gumbel noise of `philox.gumbel_row` (T = 0: plain arg-max, lowest
id on ties); `ar_logits[f, i]` is the AR head's prediction FOR position i (the caller aligns it).
"""
import numpy as np

from . import MASKED, COMMITTED, SCAFFOLD  # noqa: F401
from .philox import gumbel_row

DRAFT = 3


def ss_draft(logits, tokens, state, seeds, temperature, block_idx, step):
    """Step 2: every MASKED position gets argmax(logit + T g) and the state DRAFT."""
    logits = np.asarray(logits)
    N, d, V = logits.shape
    tokens = np.array(tokens, dtype=np.int32, copy=True)
    state = np.array(state, dtype=np.uint8, copy=True)
    for f in range(N):
        for i in range(d):
            if state[f, i] != MASKED:
                continue
            s = logits[f, i].astype(np.float64)
            if temperature != 0.0:
                s = s + float(temperature) * gumbel_row(seeds[f], block_idx, step, i, V)
            tokens[f, i] = int(np.argmax(s))
            state[f, i] = DRAFT
    return tokens, state


def ss_accept(ar_logits, tokens, state, seeds, temperature, block_idx, step):
    """Step 3.  Returns dict(tokens, state, n_accepted [N], n_left [N], score_margin [N, d]).

    n_accepted counts the positions that became COMMITTED in this call (accepted drafts plus the
    replacement token, if any); n_left the positions that are MASKED afterwards.  score_margin is
    the verifier's top-1 minus top-2 score at every position it looked at (inf elsewhere)."""
    ar_logits = np.asarray(ar_logits)
    N, d, V = ar_logits.shape
    tokens = np.array(tokens, dtype=np.int32, copy=True)
    state = np.array(state, dtype=np.uint8, copy=True)
    n_accepted = np.zeros(N, dtype=np.int32)
    n_left = np.zeros(N, dtype=np.int32)
    margin = np.full((N, d), np.inf)
    for f in range(N):
        rejected = False
        for i in range(d):
            if state[f, i] != DRAFT:
                continue
            if rejected:
                state[f, i] = MASKED                # discarded draft
                continue
            s = ar_logits[f, i].astype(np.float64)
            if temperature != 0.0:
                s = s + float(temperature) * gumbel_row(seeds[f], block_idx, step, i, V)
            t = int(np.argmax(s))
            if V > 1:
                top2 = np.partition(s, V - 2)[V - 2:]
                margin[f, i] = top2[1] - top2[0]
            if t != tokens[f, i]:
                tokens[f, i] = t                    # the verifier's token replaces the draft
                rejected = True
            state[f, i] = COMMITTED
            n_accepted[f] += 1
        n_left[f] = int(np.sum(state[f] == MASKED))
    return dict(tokens=tokens, state=state, n_accepted=n_accepted, n_left=n_left, score_margin=margin)
