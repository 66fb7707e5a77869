"""GPU parity of the scene-level paths: several layers with caches of their own, the order of
Sec. 3.4 (decode the deterministic sections once, then fork), and the bounded wait of the
attention kernel's merge."""
import numpy as np
import pytest
import torch

from oracle import MASKED
from oracle.cache import ForkSet
from oracle.jmt import average_rollouts_jmt
from oracle.unmask import unmask_step
from paper_2605_23163_b200 import fdd, harness, synth

import parity_utils as pu

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _need_cuda():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    fdd.lib()


def _attn(ctx, forkset, layer, q, k, v, d, causal=False, head_dim=128):
    qd, kd, vd = harness.bf16_tensor(q), harness.bf16_tensor(k), harness.bf16_tensor(v)
    out = torch.full_like(qd, float("nan"))
    fdd.fdd_block_attn(ctx, [forkset], layer, qd, kd, vd, out, [d], 1.0 / np.sqrt(head_dim), int(causal))
    fdd.fdd_poll_status(ctx)
    return out.float().cpu().numpy().astype(np.float64)


def _oracle_attn(w, ofs, layer, q, k, v):
    return pu.attention_oracle(w, (ofs.prefix_k[layer], ofs.prefix_v[layer]),
                               (ofs.suffix_k[layer], ofs.suffix_v[layer]), q, k, v)


def test_three_layers_with_caches_of_their_own():
    # Sec. 3.3: the caches of earlier blocks are reused, layer by layer.  Three layers with distinct
    # prefix and suffix caches; two blocks; attention on every layer against that layer's oracle
    # cache; the suffix length advances only with the last layer's commit; a second fork over the
    # same buffers (the tensor maps of the freed set serve again) reads the same caches.
    L = 3
    w = synth.small_variant(synth.workload("tts"), prefix_len=700 + 29, vocab=512, n_forks=3, n_blocks=3)
    sc = w.scenes[0]
    d = sc.block_len
    ctx = harness.create_context(w, n_layers=L)
    try:
        scene = harness.GpuScene(ctx, w, 0, n_layers=L, suffix_capacity=3 * d)
        prefixes = [synth.make_prefix(w, 0, layer) for layer in range(L)]
        assert not np.array_equal(prefixes[0][0], prefixes[1][0])
        ofs = ForkSet([p[0] for p in prefixes], [p[1] for p in prefixes], sc.n_forks, scene.seeds)
        for block in range(2):
            per_layer = [synth.make_qkv(w, 0, layer, block, 0) for layer in range(L)]
            for layer in (2, 0, 1):                        # any order: a layer reads its own caches only
                q, k, v = per_layer[layer]
                got = _attn(ctx, scene.forkset, layer, q, k, v, d)
                pu.assert_attention_close(got, _oracle_attn(w, ofs, layer, q, k, v))
            for layer in range(L):
                _, k, v = per_layer[layer]
                fdd.fdd_kv_commit(ctx, [scene.forkset], layer, harness.bf16_tensor(k), harness.bf16_tensor(v), [d],
                                  1 if layer == L - 1 else 0)
                # every layer of a block is written at the same place: the length moves with the last one
                assert fdd.fdd_forkset_suffix_len(scene.forkset) == ((block + 1) * d if layer == L - 1 else block * d)
                ofs.kv_commit(layer, k, v)
        fdd.fdd_poll_status(ctx)
        for layer in range(L):                             # the bytes landed in the right layer's buffer
            sk = scene.suffix_k[layer].view(torch.int16).cpu().numpy().view(np.uint16)
            for f in range(sc.n_forks):
                assert np.array_equal(sk[f, :, :2 * d].transpose(1, 0, 2), ofs.suffix_k[layer][f])
        # free, fork again over the same buffers, put the two blocks back, and read every layer
        scene.free()
        again = fdd.fdd_fork(ctx, scene.prefix_k, scene.prefix_v, None, sc.prefix_len, scene.prefix_capacity,
                             sc.n_forks, scene.seeds, scene.suffix_k, scene.suffix_v, scene.suffix_capacity)
        assert fdd.fdd_forkset_suffix_len(again) == 0
        for block in range(2):
            for layer in range(L):
                _, k, v = synth.make_qkv(w, 0, layer, block, 0)
                fdd.fdd_kv_commit(ctx, [again], layer, harness.bf16_tensor(k), harness.bf16_tensor(v), [d],
                                  1 if layer == L - 1 else 0)
        for layer in range(L):
            q, k, v = synth.make_qkv(w, 0, layer, 2, 1)
            got = _attn(ctx, again, layer, q, k, v, d)
            pu.assert_attention_close(got, _oracle_attn(w, ofs, layer, q, k, v))
        with pytest.raises(fdd.FddError) as ei:
            fdd.fdd_block_attn(ctx, [again], L, harness.bf16_tensor(q), harness.bf16_tensor(k), harness.bf16_tensor(v),
                               torch.empty_like(harness.bf16_tensor(q)), [d], 0.1, 0)
        assert ei.value.status == fdd.FDD_ERR_SHAPE
    finally:
        fdd.fdd_destroy(ctx)


def _decode_block_both(ctx, w, forkset, ofs, block, n, seeds, temperature, sample=None):
    """One block loop on the GPU and in the oracle, step by step from the oracle's state; returns
    the final tokens / state and the last step's K/V."""
    sc = w.scenes[0]
    tokens, state = synth.make_block_template(w, 0, block)
    tokens, state = tokens[:n].copy(), state[:n].copy()
    step, ambiguous = 0, 0
    k = v = None
    while np.any(state == MASKED):
        q, k, v = (x[:n] for x in synth.make_qkv(w, 0, 0, block, step))
        got_attn = _attn(ctx, forkset, 0, q, k, v, sc.block_len)
        pu.assert_attention_close(got_attn, _oracle_attn(w, ofs, 0, q, k, v))
        logits = synth.make_logits(w, 0, block, step, rows="all")[:n]
        tok_d = torch.from_numpy(tokens).cuda()
        st_d = torch.from_numpy(state).cuda()
        n_c = torch.zeros(n, dtype=torch.int32, device="cuda")
        n_l = torch.zeros(n, dtype=torch.int32, device="cuda")
        conf = torch.zeros(tokens.shape, dtype=torch.float32, device="cuda")
        fdd.fdd_unmask(ctx, [forkset], harness.logits_tensor(w, logits), tok_d, st_d, [sc.block_len], w.threshold,
                       temperature, block, step, n_c, n_l, conf)
        fdd.fdd_poll_status(ctx)
        got = dict(tokens=tok_d.cpu().numpy(), state=st_d.cpu().numpy(), n_committed=n_c.cpu().numpy(),
                   n_left=n_l.cpu().numpy(), conf=conf.cpu().numpy())
        ref = unmask_step(pu.widen_logits(w, logits), tokens, state, seeds, w.threshold, temperature, block, step)
        ambiguous += len(pu.compare_unmask(got, ref, tokens, state, w.threshold)["ambiguous_forks"])
        tokens, state = ref["tokens"], ref["state"]
        step += 1
        assert step <= sc.block_len
    assert ambiguous <= 2
    return tokens, state, k, v


@pytest.mark.parametrize("paged", [False, True])
def test_scene_decodes_deterministic_blocks_once_then_forks(paged):
    # Sec. 3.4: three greedy blocks by one rollout, each committed to the shared prefix itself; then
    # eight rollouts forked from that cache (nothing copied) decode three sampled blocks with private
    # suffixes; their trajectories are interpolated and averaged.  Every attention and unmasking step
    # is held against the oracle, which does the same thing on arrays.
    base = synth.workload("tts")
    P = 64 * 9 + 17 if paged else 4096
    sc = synth.Scene(prefix_len=P, n_forks=8, block_len=32, n_scaffold=10, n_blocks=6)
    w = synth.Workload("scene", base.n_q_heads, base.n_kv_heads, base.head_dim, 2048 * 5 + 1024, "bf16", "peaked",
                       0.9, 1.0, (sc,), page_tokens=64 if paged else 0, seed=41)
    d, N = sc.block_len, sc.n_forks
    ctx = harness.create_context(w)
    try:
        pk, pv = synth.make_prefix(w, 0)
        cap_tokens = P + 3 * d
        if paged:
            n_pages = (cap_tokens + 63) // 64
            pool = n_pages + 2
            ids = synth.page_order(w, 0, n_pages, pool)
            table = torch.from_numpy(ids).cuda()
            dk = harness.pack_prefix_paged(pk, 64, ids, pool)
            dv = harness.pack_prefix_paged(pv, 64, ids, pool)
            capacity = pool
        else:
            table = None
            dk = harness.pack_prefix_contiguous(pk, cap_tokens)
            dv = harness.pack_prefix_contiguous(pv, cap_tokens)
            capacity = cap_tokens
        seeds = synth.fork_seeds(w, 0)
        shape1 = (1, w.n_kv_heads, d, w.head_dim)
        s1k, s1v = (torch.zeros(shape1, dtype=torch.bfloat16, device="cuda") for _ in range(2))
        one = fdd.fdd_fork(ctx, [dk], [dv], table, P, capacity, 1, seeds[:1], [s1k], [s1v], d)
        o_one = ForkSet([pk], [pv], 1, seeds[:1])
        finished = []
        for block in range(3):                             # the deterministic sections: greedy, one rollout
            tokens, state, k, v = _decode_block_both(ctx, w, one, o_one, block, 1, seeds[:1], 0.0)
            finished.append((tokens, state))
            fdd.fdd_prefix_extend(ctx, [one], 0, harness.bf16_tensor(k), harness.bf16_tensor(v), [d], 1)
            o_one.extend_prefix(0, k, v)
            assert fdd.fdd_forkset_prefix_len(one) == P + (block + 1) * d
        fdd.fdd_poll_status(ctx)
        assert fdd.fdd_forkset_suffix_len(one) == 0
        if not paged:                                      # the contiguous cache is full now (the page pool has spare pages)
            with pytest.raises(fdd.FddError) as ei:
                fdd.fdd_prefix_extend(ctx, [one], 0, harness.bf16_tensor(k), harness.bf16_tensor(v), [d], 1)
            assert ei.value.status == fdd.FDD_ERR_CAPACITY
        P2 = fdd.fdd_forkset_prefix_len(one)
        # fork: same cache buffers, longer prefix
        shapeN = (N, w.n_kv_heads, 3 * d, w.head_dim)
        sNk, sNv = (torch.zeros(shapeN, dtype=torch.bfloat16, device="cuda") for _ in range(2))
        many = fdd.fdd_fork(ctx, [dk], [dv], table, P2, capacity, N, seeds, [sNk], [sNv], 3 * d)
        o_many = o_one.fork(N, seeds)
        with pytest.raises(fdd.FddError) as ei:            # only a set of one rollout extends the prefix
            fdd.fdd_prefix_extend(ctx, [many], 0, harness.bf16_tensor(k), harness.bf16_tensor(v), [d], 1)
        assert ei.value.status == fdd.FDD_ERR_STATE
        traj_tokens, traj_state = [], []
        for block in range(3, 6):                          # the trajectory section: sampled, N rollouts
            tokens, state, k, v = _decode_block_both(ctx, w, many, o_many, block, N, seeds, w.temperature)
            traj_tokens.append(tokens)
            traj_state.append(state)
            fdd.fdd_kv_commit(ctx, [many], 0, harness.bf16_tensor(k), harness.bf16_tensor(v), [d], 1)
            o_many.kv_commit(0, k, v)
        assert fdd.fdd_forkset_suffix_len(many) == 3 * d
        # rollouts differ (independent draws) although they share every cached token before the fork
        assert len({tuple(t.tolist()) for t in np.concatenate(traj_tokens, axis=1)}) > 1
        traj = synth.tokens_to_trajectory(w, np.concatenate(traj_tokens, axis=1), np.concatenate(traj_state, axis=1))
        out = torch.zeros((20, 2), dtype=torch.float32, device="cuda")
        fdd.fdd_average_rollouts_jmt(ctx, torch.from_numpy(traj).cuda(), N, w.waypoints, 20, out)
        fdd.fdd_poll_status(ctx)
        ref = average_rollouts_jmt(traj, 20)
        assert np.allclose(out.cpu().numpy(), ref, rtol=1e-5, atol=1e-5 * np.abs(ref).max())
    finally:
        fdd.fdd_destroy(ctx)


def test_merge_wait_that_runs_out_is_reported_and_the_context_recovers():
    # One rollout, one KV head, head dimension 64 over a 10000-token prefix: a single unit of work cut
    # into about ten pieces, whose holders wait for one another before they merge.  With a wait limit
    # of one clock the first CTA to finish gives up at once: the launch still ends, the status word
    # says FDD_ERR_DEVICE_TIMEOUT, reading it puts the counters back in order, and the next call on
    # the same context (with the default limit again) matches the oracle.
    sc = synth.Scene(prefix_len=10000, n_forks=1, block_len=16, n_scaffold=4, n_blocks=1)
    w = synth.Workload("d64_wait", 4, 1, 64, 256, "f32", "normal_sigma2", 0.9, 0.0, (sc,), qkv_sigma=0.35, seed=77)
    ctx = harness.create_context(w)
    try:
        scene = harness.GpuScene(ctx, w, 0)
        pk, pv = synth.make_prefix(w, 0)
        ofs = ForkSet([pk], [pv], 1, scene.seeds)
        q, k, v = synth.make_qkv(w, 0, 0, 0, 0)
        fdd.fdd_set_merge_wait_limit(ctx, 1)
        qd, kd, vd = harness.bf16_tensor(q), harness.bf16_tensor(k), harness.bf16_tensor(v)
        out = torch.full_like(qd, float("nan"))
        fdd.fdd_block_attn(ctx, [scene.forkset], 0, qd, kd, vd, out, [sc.block_len], 0.125, 0)
        with pytest.raises(fdd.FddError) as ei:
            fdd.fdd_poll_status(ctx)
        assert ei.value.status == fdd.FDD_ERR_DEVICE_TIMEOUT
        fdd.fdd_poll_status(ctx)                           # read and cleared
        with pytest.raises(fdd.FddError):
            fdd.fdd_set_merge_wait_limit(ctx, 0)
        fdd.fdd_set_merge_wait_limit(ctx, 4_000_000_000)
        for _ in range(2):
            got = _attn(ctx, scene.forkset, 0, q, k, v, sc.block_len, head_dim=64)
            pu.assert_attention_close(got, _oracle_attn(w, ofs, 0, q, k, v))
    finally:
        fdd.fdd_destroy(ctx)


def test_library_block_loop_matches_the_oracle_loop():
    # Sec. 3.3: fdd_decode_block runs the denoising loop of a block by itself (gated attention on
    # every layer, unmasking, counts to the host, one step ahead) and commits the block's K/V when no
    # MASK is left.  Two layers with caches of their own, two blocks in a row (the second reads what
    # the first committed).  The oracle runs its own loop on the same inputs: the number of steps,
    # the final tokens and state, the attention output of every step for the rollouts that still
    # decoded, and the committed bytes must agree; rollouts that had finished are never written.
    from oracle.decode import decode_block
    L = 2
    w = synth.small_variant(synth.workload("tts"), prefix_len=300 + 11, vocab=2048, n_forks=5, n_blocks=2)
    sc = w.scenes[0]
    N, d = sc.n_forks, sc.block_len
    scale = 1.0 / np.sqrt(w.head_dim)
    ctx = harness.create_context(w, n_layers=L)
    try:
        scene = harness.GpuScene(ctx, w, 0, n_layers=L, suffix_capacity=2 * d)
        prefixes = [synth.make_prefix(w, 0, layer) for layer in range(L)]
        ofs = ForkSet([p[0] for p in prefixes], [p[1] for p in prefixes], N, scene.seeds)
        for block in range(2):
            tokens0, state0 = synth.make_block_template(w, 0, block)
            steps_in = d                                   # a block never needs more steps than it has positions
            host = [dict(qkv=[synth.make_qkv(w, 0, layer, block, t) for layer in range(L)],
                         logits=synth.make_logits(w, 0, block, t, rows="all")) for t in range(steps_in)]
            inputs = lambda t: dict(q=[x[0] for x in host[t]["qkv"]], k=[x[1] for x in host[t]["qkv"]],
                                    v=[x[2] for x in host[t]["qkv"]], logits=host[t]["logits"])
            ref = decode_block(ofs, inputs, tokens0, state0, w.threshold, w.temperature, block, scale)
            dq = [[harness.bf16_tensor(x[0]) for x in h["qkv"]] for h in host]
            dk = [[harness.bf16_tensor(x[1]) for x in h["qkv"]] for h in host]
            dv = [[harness.bf16_tensor(x[2]) for x in h["qkv"]] for h in host]
            dout = [[torch.full_like(q_, float("nan")) for q_ in per] for per in dq]
            dlg = [harness.logits_tensor(w, h["logits"]) for h in host]
            tokens = torch.from_numpy(tokens0).cuda()
            state = torch.from_numpy(state0).cuda()
            n_c = torch.zeros(N, dtype=torch.int32, device="cuda")
            n_l = torch.zeros(N, dtype=torch.int32, device="cuda")
            steps, left = fdd.fdd_decode_block(ctx, [scene.forkset], L, steps_in, dq, dk, dv, dout, dlg, tokens, state,
                                               [d], scale, 0, w.threshold, w.temperature, block, 1, n_c, n_l)
            fdd.fdd_poll_status(ctx)
            assert left == 0 and steps == ref["steps"] and 2 <= steps < d
            assert np.array_equal(state.cpu().numpy(), ref["state"]) and not np.any(ref["state"] == MASKED)
            assert np.array_equal(tokens.cpu().numpy(), ref["tokens"])
            assert fdd.fdd_forkset_suffix_len(scene.forkset) == (block + 1) * d
            # attention of every step: who still decoded on entry follows from the oracle's commits
            masked_left = (state0 == MASKED).sum(axis=1)
            for t in range(steps + 1):                     # the step after the last one was issued ahead and must do nothing
                decoding = np.nonzero(masked_left > 0)[0] if t < steps else np.zeros(0, dtype=int)
                for layer in range(L):
                    got = dout[t][layer].float().cpu().numpy().astype(np.float64).reshape(N, d, w.n_q_heads, w.head_dim)
                    if t < steps:
                        pu.assert_attention_close(got[decoding], ref["attn"][t][layer][decoding])
                    idle = np.setdiff1d(np.arange(N), decoding)
                    assert np.all(np.isnan(got[idle])), "attention wrote rows of a rollout that had finished"
                if t < steps:
                    masked_left = masked_left - ref["committed_per_step"][t]
            for layer in range(L):                         # the committed bytes (the oracle's loop commits too)
                sk = scene.suffix_k[layer].view(torch.int16).cpu().numpy().view(np.uint16)
                for f in range(N):
                    assert np.array_equal(sk[f, :, :(block + 1) * d].transpose(1, 0, 2), ofs.suffix_k[layer][f])
        # a loop that is cut short says so and commits nothing
        tokens0, state0 = synth.make_block_template(w, 0, 0)
        tokens, state = torch.from_numpy(tokens0).cuda(), torch.from_numpy(state0).cuda()
        before = fdd.fdd_forkset_suffix_len(scene.forkset)
        steps, left = fdd.fdd_decode_block(ctx, [scene.forkset], L, 1, dq[:1], dk[:1], dv[:1], dout[:1], dlg[:1], tokens, state,
                                           [d], scale, 0, w.threshold, w.temperature, 0, 1, n_c, n_l)
        fdd.fdd_poll_status(ctx)
        assert steps == 1 and left == int((state.cpu().numpy() == MASKED).sum()) > 0
        assert fdd.fdd_forkset_suffix_len(scene.forkset) == before
        # argument errors come back before anything is issued
        launches = fdd.fdd_launch_count(ctx)
        for bad in (dict(n_layers=L + 1), dict(max_steps=0)):
            with pytest.raises(fdd.FddError) as ei:
                fdd.fdd_decode_block(ctx, [scene.forkset], bad.get("n_layers", L), bad.get("max_steps", 1), dq[:1], dk[:1], dv[:1],
                                     dout[:1], dlg[:1], tokens, state, [d], scale, 0, w.threshold, w.temperature, 0, 1, n_c, n_l)
            assert ei.value.status == fdd.FDD_ERR_INVALID_ARG
        assert fdd.fdd_launch_count(ctx) == launches
    finally:
        fdd.fdd_destroy(ctx)


def test_library_block_loop_with_more_scenes_than_one_unmask_launch_takes():
    # Eighteen small scenes (different rollouts, block lengths and prefix lengths) in one
    # fdd_decode_block call: the unmasking step splits them into two launches, whose counts must all
    # reach the loop's host buffer at the right place.  Every scene against the oracle's own loop.
    from oracle.decode import decode_block
    base = synth.workload("serving_mix")
    rng = np.random.default_rng(7)
    scenes = tuple(synth.Scene(int(rng.integers(1, 200)), int(rng.integers(1, 4)), int(rng.choice([16, 32])),
                               int(rng.integers(3, 9)), 1) for _ in range(18))
    w = synth.Workload("mix_loop", base.n_q_heads, base.n_kv_heads, base.head_dim, 512, "bf16", "peaked", 0.9, 1.0,
                       scenes, page_tokens=64, seed=23)
    scale = 1.0 / np.sqrt(w.head_dim)
    d_max = max(sc.block_len for sc in scenes)
    ctx = harness.create_context(w)
    try:
        gs = [harness.GpuScene(ctx, w, i, suffix_capacity=sc.block_len) for i, sc in enumerate(scenes)]
        refs, host_steps = [], [[] for _ in range(d_max)]
        tokens0, state0 = [], []
        for i, sc in enumerate(scenes):
            pk, pv = synth.make_prefix(w, i)
            ofs = ForkSet([pk], [pv], sc.n_forks, gs[i].seeds)
            t0, s0 = synth.make_block_template(w, i, 0)
            per_step = [dict(qkv=synth.make_qkv(w, i, 0, 0, t), logits=synth.make_logits(w, i, 0, t, rows="all"))
                        for t in range(d_max)]
            inputs = lambda t, ps=per_step: dict(q=[ps[t]["qkv"][0]], k=[ps[t]["qkv"][1]], v=[ps[t]["qkv"][2]],
                                                 logits=ps[t]["logits"])
            refs.append(decode_block(ofs, inputs, t0, s0, w.threshold, w.temperature, 0, scale, want_attention=False))
            for t in range(d_max):
                host_steps[t].append(per_step[t])
            tokens0.append(t0.reshape(-1)); state0.append(s0.reshape(-1))
        pack = lambda xs: np.concatenate([np.asarray(x).reshape(-1) for x in xs])
        dq = [[harness.bf16_tensor(pack([p["qkv"][0] for p in host_steps[t]]))] for t in range(d_max)]
        dk = [[harness.bf16_tensor(pack([p["qkv"][1] for p in host_steps[t]]))] for t in range(d_max)]
        dv = [[harness.bf16_tensor(pack([p["qkv"][2] for p in host_steps[t]]))] for t in range(d_max)]
        dout = [[torch.empty_like(x[0])] for x in dq]
        dlg = [harness.logits_tensor(w, pack([p["logits"] for p in host_steps[t]])) for t in range(d_max)]
        tokens = torch.from_numpy(np.concatenate(tokens0)).cuda()
        state = torch.from_numpy(np.concatenate(state0)).cuda()
        N = sum(sc.n_forks for sc in scenes)
        n_c = torch.zeros(N, dtype=torch.int32, device="cuda")
        n_l = torch.zeros(N, dtype=torch.int32, device="cuda")
        steps, left = fdd.fdd_decode_block(ctx, [g.forkset for g in gs], 1, d_max, dq, dk, dv, dout, dlg, tokens, state,
                                           [sc.block_len for sc in scenes], scale, 0, w.threshold, w.temperature, 0, 1,
                                           n_c, n_l)
        fdd.fdd_poll_status(ctx)
        assert left == 0 and steps == max(r["steps"] for r in refs)
        got_tok, got_st = tokens.cpu().numpy(), state.cpu().numpy()
        off = 0
        for sc, ref, g in zip(scenes, refs, gs):
            n = sc.n_forks * sc.block_len
            assert np.array_equal(got_st[off:off + n].reshape(ref["state"].shape), ref["state"])
            assert np.array_equal(got_tok[off:off + n].reshape(ref["tokens"].shape), ref["tokens"])
            assert fdd.fdd_forkset_suffix_len(g.forkset) == sc.block_len
            off += n
    finally:
        fdd.fdd_destroy(ctx)
