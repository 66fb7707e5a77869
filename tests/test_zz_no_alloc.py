"""fdd_unmask_static: the unmasking step for callers that are not allowed to allocate.

A planning loop that has finished its start-up phase, or a component that only receives
pre-allocated buffers, cannot go through fdd_create / fdd_fork, because both allocate device
memory.  fdd_unmask_static needs neither: its scratch is a fixed array inside the library.  This
test calls it through the C ABI twice in a row (the second call sees the first call's leftovers in
the shared scratch) and requires exactly the results of the regular entry point: identical tokens,
states and counters, confidences within the tolerance the other unmask tests use.  Both calls are
also held against the CPU oracle, under the same rules as every other unmask parity test.

Collected last on purpose, so that a run that stops at the first failure has already run every
other test; it also passes when run on its own in a fresh process.
"""
import numpy as np
import pytest
import torch

from oracle.unmask import unmask_step
from paper_2605_23163_b200 import fdd, harness, synth
from parity_utils import CONF_TOL, compare_unmask, widen_logits

pytestmark = pytest.mark.gpu


def _regular(w, logits, tokens, state, seeds, step):
    ctx = harness.create_context(w)
    try:
        scene = harness.GpuScene(ctx, w, 0)
        tok = torch.from_numpy(tokens.copy()).cuda()
        st = torch.from_numpy(state.copy()).cuda()
        n = tokens.shape[0]
        nc = torch.zeros(n, dtype=torch.int32, device="cuda")
        nl = torch.zeros(n, dtype=torch.int32, device="cuda")
        conf = torch.zeros(tokens.shape, dtype=torch.float32, device="cuda")
        fdd.fdd_unmask(ctx, [scene.forkset], harness.logits_tensor(w, logits), tok, st, [tokens.shape[1]],
                       w.threshold, w.temperature, 0, step, nc, nl, conf)
        fdd.fdd_poll_status(ctx)
        return tok.cpu().numpy(), st.cpu().numpy(), nc.cpu().numpy(), nl.cpu().numpy(), conf.cpu().numpy()
    finally:
        fdd.fdd_destroy(ctx)


def _static(w, logits, tokens, state, seeds, step):
    tok = torch.from_numpy(tokens.copy()).cuda()
    st = torch.from_numpy(state.copy()).cuda()
    n = tokens.shape[0]
    nc = torch.zeros(n, dtype=torch.int32, device="cuda")
    nl = torch.zeros(n, dtype=torch.int32, device="cuda")
    conf = torch.zeros(tokens.shape, dtype=torch.float32, device="cuda")
    seeds_d = torch.from_numpy(np.asarray(seeds, dtype=np.uint64).view(np.int64)).cuda()
    dtype = fdd.FDD_LOGITS_BF16 if w.logits_dtype == "bf16" else fdd.FDD_LOGITS_F32
    fdd.fdd_unmask_static(harness.logits_tensor(w, logits), dtype, n, tokens.shape[1], w.vocab, tok, st,
                          seeds_d, w.threshold, w.temperature, 0, step, nc, nl, conf)
    torch.cuda.synchronize()
    return tok.cpu().numpy(), st.cpu().numpy(), nc.cpu().numpy(), nl.cpu().numpy(), conf.cpu().numpy()


def _same(a, b):
    for x, y in zip(a[:4], b[:4]):
        assert np.array_equal(x, y)
    assert np.array_equal(np.isnan(a[4]), np.isnan(b[4]))
    assert np.nanmax(np.abs(a[4] - b[4])) <= CONF_TOL


def _matches_oracle(w, got, logits, tokens, state, seeds, step):
    ref = unmask_step(widen_logits(w, logits), tokens, state, seeds, w.threshold, w.temperature, 0, step)
    res = compare_unmask(dict(tokens=got[0], state=got[1], n_committed=got[2], n_left=got[3], conf=got[4]),
                         ref, tokens, state, w.threshold)
    assert len(res["ambiguous_forks"]) <= 1


def test_static_entry_matches_regular_entry_twice():
    assert torch.cuda.is_available()
    # first call: several chunks per row, noisy arg-max, 4 rollouts
    w1 = synth.small_variant(synth.workload("tts"), prefix_len=64, vocab=8192 * 3 + 520, n_forks=4, n_blocks=1)
    tokens, state = synth.make_block_template(w1, 0, 0)
    seeds = synth.fork_seeds(w1, 0)
    logits = synth.make_logits(w1, 0, 0, 0, rows="all")
    got = _static(w1, logits, tokens, state, seeds, 0)
    _same(got, _regular(w1, logits, tokens, state, seeds, 0))
    _matches_oracle(w1, got, logits, tokens, state, seeds, 0)
    # second call right after, different shape and dtype: the shared scratch still holds the first
    # call's records, which must not leak into this result
    w2 = synth.workload("tiny")
    tokens, state = synth.make_block_template(w2, 0, 0)
    seeds = synth.fork_seeds(w2, 0)
    logits = synth.make_logits(w2, 0, 0, 3, rows="all")
    got = _static(w2, logits, tokens, state, seeds, 3)
    _same(got, _regular(w2, logits, tokens, state, seeds, 3))
    _matches_oracle(w2, got, logits, tokens, state, seeds, 3)


def test_static_entry_rejects_oversize_and_bad_arguments():
    assert torch.cuda.is_available()
    t = torch.zeros(16, dtype=torch.int32, device="cuda")
    with pytest.raises(fdd.FddError) as ei:      # 64 * 128 rows x 19 chunks > 65536 records
        fdd.fdd_unmask_static(t, fdd.FDD_LOGITS_BF16, 64, 128, 151936, t, t, t, 0.9, 0.0, 0, 0, t, t)
    assert ei.value.status == fdd.FDD_ERR_CAPACITY and "exceeds the fixed scratch" in str(ei.value)
    with pytest.raises(fdd.FddError) as ei:      # 128 x 128 rows: few records (vocab 4096), but more rows than one call takes
        fdd.fdd_unmask_static(t, fdd.FDD_LOGITS_F32, 128, 128, 4096, t, t, t, 0.9, 0.0, 0, 0, t, t)
    assert ei.value.status == fdd.FDD_ERR_CAPACITY and "8192 rows" in str(ei.value)
    with pytest.raises(fdd.FddError) as ei:
        fdd.fdd_unmask_static(None, fdd.FDD_LOGITS_BF16, 1, 16, 64, t, t, t, 0.9, 0.0, 0, 0, t, t)
    assert ei.value.status == fdd.FDD_ERR_INVALID_ARG
    with pytest.raises(fdd.FddError) as ei:
        fdd.fdd_unmask_static(t, fdd.FDD_LOGITS_BF16, 1, 129, 64, t, t, t, 0.9, 0.0, 0, 0, t, t)
    assert ei.value.status == fdd.FDD_ERR_UNSUPPORTED
