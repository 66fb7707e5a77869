"""Confidence-threshold parallel unmasking of one block (test infrastructure).

The paper states only that Section Diffusion "iteratively unmasks value
positions" starting from the pre-filled scaffold (Sec. 3.3), that visible
tokens stay fixed in the reverse process (Sec. 3.1) and that scaffold positions
are never masked or rewritten (Sec. 3.2).  The rule below is this repository's
reading of the confidence-based parallel decoding it builds on:

for every rollout f and every position i whose state is MASKED
    s[v]   = logit[v] + temperature * g[v]          (g: Gumbel noise; none if temperature == 0)
    tok_i  = argmax_v s[v]                           (lowest v on ties)
    conf_i = softmax(logit)[tok_i]                   (noise-free probability of the chosen token)
commit set C_f = { i MASKED : conf_i > threshold };  if it is empty while
some position is MASKED, C_f = { the MASKED i with the largest conf_i }
(lowest i on ties).  For i in C_f: tokens[i] = tok_i, state[i] = COMMITTED.
Nothing else is written.  A rollout without MASKED positions is left alone.

argmax(l + T*g) draws exactly from softmax(l / T) (Gumbel-max), which is how
"sampled at non-zero temperature" (Sec. 3.4) enters.
"""
import numpy as np

from . import MASKED, COMMITTED, SCAFFOLD  # noqa: F401
from .philox import gumbel_row


def unmask_step(logits, tokens, state, seeds, threshold, temperature, block_idx, step):
    """One unmasking step.

    logits: [N, d, V] float (any dtype, widened to fp64); tokens: [N, d] int;
    state: [N, d] uint8; seeds: [N] 64-bit ints.
    Returns dict with new `tokens`, `state`, `n_committed` [N], `n_left` [N],
    `conf` [N, d] (NaN where the position was not MASKED), `choice` [N, d]
    (-1 where not MASKED), `score_margin` [N, d] (top-1 minus top-2 of s; inf
    where not MASKED) and `fallback` [N] (bool: the at-least-one rule fired).
    """
    logits = np.asarray(logits)
    N, d, V = logits.shape
    tokens = np.array(tokens, dtype=np.int32, copy=True)
    state = np.array(state, dtype=np.uint8, copy=True)
    conf = np.full((N, d), np.nan, dtype=np.float64)
    choice = np.full((N, d), -1, dtype=np.int64)
    margin = np.full((N, d), np.inf, dtype=np.float64)
    n_committed = np.zeros(N, dtype=np.int32)
    n_left = np.zeros(N, dtype=np.int32)
    fallback = np.zeros(N, dtype=bool)
    for f in range(N):
        masked = [i for i in range(d) if state[f, i] == MASKED]
        if not masked:
            continue
        for i in masked:
            l = logits[f, i].astype(np.float64)
            if temperature != 0.0:
                s = l + float(temperature) * gumbel_row(seeds[f], block_idx, step, i, V)
            else:
                s = l
            t = int(np.argmax(s))                      # numpy: first maximal index
            m = np.max(l)
            lse = m + np.log(np.sum(np.exp(l - m)))
            conf[f, i] = np.exp(l[t] - lse)
            choice[f, i] = t
            if V > 1:
                top2 = np.partition(s, V - 2)[V - 2:]
                margin[f, i] = top2[1] - top2[0]
        commit = [i for i in masked if conf[f, i] > threshold]
        if not commit:
            best = masked[0]
            for i in masked[1:]:
                if conf[f, i] > conf[f, best]:
                    best = i
            commit = [best]
            fallback[f] = True
        for i in commit:
            tokens[f, i] = choice[f, i]
            state[f, i] = COMMITTED
        n_committed[f] = len(commit)
        n_left[f] = len(masked) - len(commit)
    return dict(tokens=tokens, state=state, n_committed=n_committed, n_left=n_left,
                conf=conf, choice=choice, score_margin=margin, fallback=fallback)
