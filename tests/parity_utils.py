"""Helpers shared by the GPU parity tests: run one call on the GPU through the binding and the
same seeded inputs through the CPU oracle, and compare under the stated tolerances."""
import numpy as np
import torch

from oracle import MASKED
from oracle.attention import bf16_bits_to_f64, decode_block_attention, causal_block_attention_rows
from oracle.unmask import unmask_step
from paper_2605_23163_b200 import fdd, harness, synth

# attention: bf16 inputs, fp32 accumulation, bf16 output against the fp64 oracle
ATTN_MAX_ABS = 1e-2
ATTN_REL_L2 = 5e-3
# unmask: token ids bit-exact where the oracle's top-two score margin exceeds this
SCORE_MARGIN = 1e-3
CONF_NEAR = 1e-4          # |conf - threshold| below this: a commit flip is a rounding artefact
CONF_TOL = 5e-6           # fp32 confidence against the fp64 oracle (absolute)


def attention_gpu(ctx, scene, q_bits, k_bits, v_bits, layer=0, causal=False, scale=None):
    w = scene.w
    q = harness.bf16_tensor(q_bits)
    k = harness.bf16_tensor(k_bits)
    v = harness.bf16_tensor(v_bits)
    out = torch.full_like(q, float("nan"))
    scale = scale if scale is not None else 1.0 / np.sqrt(w.head_dim)
    fdd.fdd_block_attn(ctx, [scene.forkset], layer, q, k, v, out, [q_bits.shape[1]], scale, int(causal))
    fdd.fdd_poll_status(ctx)
    return out.float().cpu().numpy().astype(np.float64)


def attention_oracle(w, prefix_bits, suffix_bits, q_bits, k_bits, v_bits, causal=False, scale=None,
                     forks=None):
    """suffix_bits: (list of [S,Hkv,D] K bits per fork, same for V)."""
    W = bf16_bits_to_f64
    scale = scale if scale is not None else 1.0 / np.sqrt(w.head_dim)
    forks = list(range(q_bits.shape[0])) if forks is None else list(forks)
    fn = causal_block_attention_rows if causal else decode_block_attention
    return fn(W(q_bits[forks]), W(k_bits[forks]), W(v_bits[forks]), W(prefix_bits[0]), W(prefix_bits[1]),
              [W(suffix_bits[0][f]) for f in forks], [W(suffix_bits[1][f]) for f in forks], scale)


def assert_attention_close(got, ref):
    assert np.all(np.isfinite(got)), "non-finite attention output"
    max_abs = float(np.max(np.abs(got - ref)))
    rel_l2 = float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30))
    assert max_abs <= ATTN_MAX_ABS, f"max-abs {max_abs}"
    assert rel_l2 <= ATTN_REL_L2, f"rel-L2 {rel_l2}"
    return max_abs, rel_l2


def unmask_gpu(ctx, scene, logits_arr, tokens, state, threshold, temperature, block_idx, step,
               want_conf=True):
    w = scene.w
    lg = harness.logits_tensor(w, logits_arr)
    tok = torch.from_numpy(np.ascontiguousarray(tokens, dtype=np.int32)).cuda()
    st = torch.from_numpy(np.ascontiguousarray(state, dtype=np.uint8)).cuda()
    n = tokens.shape[0]
    n_comm = torch.full((n,), -7, dtype=torch.int32, device="cuda")
    n_left = torch.full((n,), -7, dtype=torch.int32, device="cuda")
    conf = torch.zeros(tokens.shape, dtype=torch.float32, device="cuda") if want_conf else None
    fdd.fdd_unmask(ctx, [scene.forkset], lg, tok, st, [tokens.shape[1]], threshold, temperature,
                   block_idx, step, n_comm, n_left, conf)
    fdd.fdd_poll_status(ctx)
    return dict(tokens=tok.cpu().numpy(), state=st.cpu().numpy(), n_committed=n_comm.cpu().numpy(),
                n_left=n_left.cpu().numpy(), conf=None if conf is None else conf.cpu().numpy())


def widen_logits(w, arr):
    return bf16_bits_to_f64(arr) if w.logits_dtype == "bf16" else arr.astype(np.float64)


def compare_unmask(got, ref, tokens_in, state_in, threshold):
    """Compare one step.  Returns dict(ambiguous_forks=set, low_margin_rows=int, rows=int).

    Bit-exact: for every MASKED row whose oracle score margin > SCORE_MARGIN the token the GPU
    would commit equals the oracle's; for every rollout that is not ambiguous (no row within
    CONF_NEAR of the threshold, no near-tie in the at-least-one pick, no low-margin row among
    its commits) tokens, states and counters are identical; inside an ambiguous rollout every
    position that is clear by itself still has to agree.  Everything that was not MASKED is
    untouched in every rollout."""
    N, d = tokens_in.shape
    keep = state_in != MASKED
    assert np.array_equal(got["tokens"][keep], tokens_in[keep]), "a non-MASKED token was rewritten"
    assert np.array_equal(got["state"][keep], state_in[keep]), "a non-MASKED state was rewritten"
    ambiguous, low_margin, rows = set(), 0, 0
    for f in range(N):
        masked = np.nonzero(state_in[f] == MASKED)[0]
        rows += len(masked)
        if len(masked) == 0:
            assert got["n_committed"][f] == 0 and got["n_left"][f] == 0
            continue
        amb = False
        confs = ref["conf"][f, masked]
        if got["conf"] is not None:
            gc = got["conf"][f]
            assert np.all(np.isnan(gc[state_in[f] != MASKED]))
            assert np.max(np.abs(gc[masked] - confs)) <= CONF_TOL, \
                f"confidence off by {np.max(np.abs(gc[masked] - confs))}"
        if np.any(np.abs(confs - threshold) < CONF_NEAR):
            amb = True
        if ref["fallback"][f] and len(masked) > 1:
            top2 = np.sort(confs)[-2:]
            if top2[1] - top2[0] < CONF_NEAR * max(top2[1], 1e-30):
                amb = True
        lm = ref["score_margin"][f, masked] <= SCORE_MARGIN
        low_margin += int(lm.sum())
        committed_ref = masked[ref["state"][f, masked] != MASKED]
        if np.any(ref["score_margin"][f, committed_ref] <= SCORE_MARGIN):
            amb = True
        if amb:
            # Even here every position that is clear by itself is held to the oracle: a confidence
            # clearly above the threshold must be committed, with the oracle's token wherever the
            # score margin allows; one clearly below may be committed only by the at-least-one rule
            # (then it is the rollout's single commit); a token written for a row with a clear
            # margin is the oracle's choice.
            ambiguous.add(f)
            for i in masked:
                clear_margin = ref["score_margin"][f, i] > SCORE_MARGIN
                committed = got["state"][f, i] != MASKED
                if committed and clear_margin:
                    assert got["tokens"][f, i] == ref["choice"][f, i], f"rollout {f} position {i}: token differs"
                if ref["conf"][f, i] > threshold + CONF_NEAR:
                    assert committed, f"rollout {f} position {i}: clear pass not committed"
                elif ref["conf"][f, i] < threshold - CONF_NEAR and committed:
                    assert got["n_committed"][f] == 1, f"rollout {f} position {i}: committed below the threshold"
            assert got["n_committed"][f] == int((got["state"][f, masked] != MASKED).sum())
            assert got["n_left"][f] == int((got["state"][f, masked] == MASKED).sum())
            continue
    return dict(ambiguous_forks=ambiguous, low_margin_rows=low_margin, rows=rows)


def scene_bits(w, scene_idx, layer=0):
    return synth.make_prefix(w, scene_idx, layer)
