"""GPU parity: every C-ABI call against the CPU fp64 oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import MASKED, COMMITTED, SCAFFOLD
from oracle.average import average_rollouts
from oracle.cache import ForkSet
from oracle.unmask import unmask_step
from paper_2605_23163_b200 import fdd, harness, synth

import parity_utils as pu

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _need_cuda():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    fdd.lib()   # fail loudly if the CUDA library is missing


def _suffix_from_oracle(fs, layer=0):
    return (fs.suffix_k[layer], fs.suffix_v[layer])


# ---------------------------------------------------------------------------------------------
# attention
# ---------------------------------------------------------------------------------------------
def _attention_case(w, n_blocks_before=0, causal=False, forks_checked=None, layer=0):
    ctx = harness.create_context(w)
    try:
        scene = harness.GpuScene(ctx, w, 0, suffix_capacity=w.scenes[0].block_len * (n_blocks_before + 1))
        pk, pv = synth.make_prefix(w, 0)
        ofs = ForkSet([pk], [pv], w.scenes[0].n_forks, scene.seeds)
        for b in range(n_blocks_before):         # fill the private suffix with earlier blocks
            _, kb, vb = synth.make_qkv(w, 0, 0, b, 0)
            fdd.fdd_kv_commit(ctx, [scene.forkset], 0, harness.bf16_tensor(kb), harness.bf16_tensor(vb),
                              [kb.shape[1]], 1)
            ofs.kv_commit(0, kb, vb)
        assert fdd.fdd_forkset_suffix_len(scene.forkset) == n_blocks_before * w.scenes[0].block_len
        q, k, v = synth.make_qkv(w, 0, 0, n_blocks_before, 0)
        got = pu.attention_gpu(ctx, scene, q, k, v, causal=causal)
        forks = list(range(q.shape[0])) if forks_checked is None else forks_checked
        ref = pu.attention_oracle(w, (pk, pv), _suffix_from_oracle(ofs), q, k, v, causal=causal, forks=forks)
        return pu.assert_attention_close(got[forks], ref)
    finally:
        fdd.fdd_destroy(ctx)


def test_attention_tiny():
    _attention_case(synth.workload("tiny"))


def test_attention_single_scene_with_suffix():
    _attention_case(synth.workload("single_scene"), n_blocks_before=2)


def test_attention_tts_all_forks():
    _attention_case(synth.workload("tts"), n_blocks_before=1)


def test_attention_tts_ragged_prefix_and_block():
    # prefix not a multiple of any tile, block of 13 positions (ragged row tile), 3 rollouts
    w = synth.workload("tts")
    sc = synth.Scene(prefix_len=1000 + 37, n_forks=3, block_len=13, n_scaffold=4, n_blocks=3)
    w = synth.Workload("ragged", w.n_q_heads, w.n_kv_heads, w.head_dim, 1024, "bf16", "peaked", 0.9, 1.0,
                       (sc,), seed=11)
    _attention_case(w, n_blocks_before=2)


def test_attention_long_prefix_sampled_forks():
    # full-size largest configuration; the oracle checks three of the 32 rollouts
    _attention_case(synth.workload("long_prefix"), forks_checked=[0, 13, 31])


def test_attention_long_prefix_two_rollouts_left_units_cut_into_many_pieces():
    # late in a block only a few rollouts still decode: at the largest configuration two live
    # rollouts make 16 units of 129 key tiles on 148 CTAs, so every unit is cut into about ten
    # pieces (more than the merge folds in at once); causal and bidirectional
    w = synth.workload("long_prefix")
    sc = w.scenes[0]
    ctx = harness.create_context(w)
    try:
        scene = harness.GpuScene(ctx, w, 0)
        pk, pv = synth.make_prefix(w, 0)
        empty = ([np.zeros((0, w.n_kv_heads, w.head_dim), dtype=np.uint16)] * sc.n_forks,) * 2
        q, k, v = synth.make_qkv(w, 0, 0, 0, 3)
        qd, kd, vd = harness.bf16_tensor(q), harness.bf16_tensor(k), harness.bf16_tensor(v)
        live = [5, 30]
        gate = torch.zeros(sc.n_forks, dtype=torch.int32, device="cuda")
        gate[live] = 2
        for causal in (False, True):
            out = torch.full_like(qd, float("nan"))
            fdd.fdd_block_attn_gated(ctx, [scene.forkset], 0, qd, kd, vd, out, [sc.block_len],
                                     1.0 / np.sqrt(w.head_dim), int(causal), gate)
            fdd.fdd_poll_status(ctx)
            got = out.float().cpu().numpy().astype(np.float64).reshape(q.shape)
            ref = pu.attention_oracle(w, (pk, pv), empty, q, k, v, causal=causal, forks=live)
            pu.assert_attention_close(got[live], ref)
            rest = np.setdiff1d(np.arange(sc.n_forks), live)
            assert np.all(np.isnan(got[rest]))
    finally:
        fdd.fdd_destroy(ctx)


@pytest.mark.parametrize("prefix_len", [2100, 4096, 10000])
def test_attention_head_dim_64_single_unit_cut_into_pieces(prefix_len):
    # head dimension 64 with one rollout and one KV head: a single unit of 18 / 33 / 80 key tiles,
    # cut into 2 / 4 / 10 pieces, so each branch of the merge (by piece count) runs at D = 64 too
    sc = synth.Scene(prefix_len=prefix_len, n_forks=1, block_len=16, n_scaffold=4, n_blocks=1)
    w = synth.Workload("d64_split", 4, 1, 64, 256, "f32", "normal_sigma2", 0.9, 0.0, (sc,), qkv_sigma=0.35, seed=50 + prefix_len)
    _attention_case(w)
    _attention_case(w, causal=True)


def test_attention_no_prefix_and_single_position():
    w = synth.workload("tiny")
    sc = synth.Scene(prefix_len=0, n_forks=2, block_len=1, n_scaffold=0, n_blocks=2)
    w = synth.Workload("degenerate", 4, 1, 64, 64, "f32", "normal_sigma2", 0.9, 0.0, (sc,), qkv_sigma=0.5, seed=12)
    _attention_case(w, n_blocks_before=0)       # a single key: output == that value row
    _attention_case(w, n_blocks_before=1)


def test_attention_causal_in_block():
    w = synth.small_variant(synth.workload("tts"), prefix_len=300, vocab=512, n_forks=2, n_blocks=2)
    _attention_case(w, n_blocks_before=1, causal=True)


def test_attention_paged_prefix():
    w = synth.workload("serving_mix")
    sc = synth.Scene(prefix_len=64 * 9 + 17, n_forks=4, block_len=16, n_scaffold=5, n_blocks=2)
    w = synth.Workload("paged", w.n_q_heads, w.n_kv_heads, w.head_dim, 1024, "bf16", "peaked", 0.9, 1.0,
                       (sc,), page_tokens=64, seed=13)
    _attention_case(w, n_blocks_before=1)


def test_attention_many_scenes_one_call():
    # a ragged serving batch in ONE call: scenes differ in prefix length, rollouts and block length;
    # paged prefix with shuffled physical pages; every scene has an earlier block in its suffix
    base = synth.workload("serving_mix")
    scenes = (synth.Scene(64 * 5 + 9, 4, 16, 5, 2), synth.Scene(64 * 21, 1, 32, 10, 2),
              synth.Scene(700, 3, 64, 19, 2), synth.Scene(130, 2, 32, 10, 2), synth.Scene(1, 1, 16, 5, 2))
    w = synth.Workload("mix_small", base.n_q_heads, base.n_kv_heads, base.head_dim, 1024, "bf16", "peaked", 0.9, 1.0,
                       scenes, page_tokens=64, seed=17)
    ctx = harness.create_context(w)
    try:
        gs, refs, qs, ks, vs = [], [], [], [], []
        for i, sc in enumerate(scenes):
            g = harness.GpuScene(ctx, w, i, suffix_capacity=2 * sc.block_len)
            pk, pv = synth.make_prefix(w, i)
            ofs = ForkSet([pk], [pv], sc.n_forks, g.seeds)
            _, kb, vb = synth.make_qkv(w, i, 0, 0, 0)
            fdd.fdd_kv_commit(ctx, [g.forkset], 0, harness.bf16_tensor(kb), harness.bf16_tensor(vb), [sc.block_len], 1)
            ofs.kv_commit(0, kb, vb)
            q, k, v = synth.make_qkv(w, i, 0, 1, 0)
            refs.append(pu.attention_oracle(w, (pk, pv), _suffix_from_oracle(ofs), q, k, v))
            gs.append(g); qs.append(q); ks.append(k); vs.append(v)
        pack = lambda xs: harness.bf16_tensor(np.concatenate([x.reshape(-1) for x in xs]))
        qd, kd, vd = pack(qs), pack(ks), pack(vs)
        out = torch.full_like(qd, float("nan"))
        fdd.fdd_block_attn(ctx, [g.forkset for g in gs], 0, qd, kd, vd, out, [sc.block_len for sc in scenes],
                           1.0 / np.sqrt(w.head_dim), 0)
        fdd.fdd_poll_status(ctx)
        got = out.float().cpu().numpy().astype(np.float64)
        off = 0
        for sc, ref in zip(scenes, refs):
            n = ref.size
            pu.assert_attention_close(got[off:off + n].reshape(ref.shape), ref)
            off += n
        assert off == got.size
    finally:
        fdd.fdd_destroy(ctx)


def test_attention_many_short_units_per_cta():
    # Hundreds of units of two to four key tiles each, so that every CTA's range holds half a dozen
    # items: whole units, pieces at both ends, and, at the borders between the scenes, the change
    # between units with two query tiles (256 stacked rows) and units with one.  The items of a range
    # follow one another without a barrier of the whole CTA; every output row is compared.
    base = synth.workload("long_prefix")
    scenes = (synth.Scene(130, 48, 64, 19, 1), synth.Scene(70, 40, 16, 5, 1), synth.Scene(300, 24, 32, 10, 1),
              synth.Scene(129, 9, 64, 19, 1))
    w = synth.Workload("short_units", base.n_q_heads, base.n_kv_heads, base.head_dim, 1024, "bf16", "peaked", 0.9, 1.0,
                       scenes, seed=23)
    ctx = harness.create_context(w)
    try:
        gs, refs, qs, ks, vs = [], [], [], [], []
        for i, sc in enumerate(scenes):
            gs.append(harness.GpuScene(ctx, w, i))
            pk, pv = synth.make_prefix(w, i)
            q, k, v = synth.make_qkv(w, i, 0, 0, 0)
            empty = ([np.zeros((0, w.n_kv_heads, w.head_dim), dtype=np.uint16)] * sc.n_forks,) * 2
            refs.append(pu.attention_oracle(w, (pk, pv), empty, q, k, v))
            qs.append(q); ks.append(k); vs.append(v)
        pack = lambda xs: harness.bf16_tensor(np.concatenate([x.reshape(-1) for x in xs]))
        qd, kd, vd = pack(qs), pack(ks), pack(vs)
        for rep in range(2):                 # (the second call finds the counters of the cut units as the first left them)
            out = torch.full_like(qd, float("nan"))
            n0 = fdd.fdd_launch_count(ctx)
            fdd.fdd_block_attn(ctx, [g.forkset for g in gs], 0, qd, kd, vd, out, [sc.block_len for sc in scenes],
                               1.0 / np.sqrt(w.head_dim), 0)
            fdd.fdd_poll_status(ctx)
            assert fdd.fdd_launch_count(ctx) - n0 == 1
            got = out.float().cpu().numpy().astype(np.float64)
            off = 0
            for ref in refs:
                pu.assert_attention_close(got[off:off + ref.size].reshape(ref.shape), ref)
                off += ref.size
            assert off == got.size
    finally:
        fdd.fdd_destroy(ctx)


def test_attention_gated_rollouts_are_skipped_and_the_rest_is_unchanged():
    # fdd_block_attn_gated: rollouts whose gate entry is 0 sit the call out (their rows of out keep
    # what was there), every other rollout gets what the ungated call gives, whatever the mix:
    # some rollouts of a scene, a whole scene, everything, nothing.  The gate is the n_left array of
    # an unmask step, so any non-zero value counts as "still decoding".
    base = synth.workload("serving_mix")
    scenes = (synth.Scene(64 * 9 + 5, 5, 32, 10, 1), synth.Scene(64 * 30, 2, 64, 19, 1),
              synth.Scene(333, 37, 16, 5, 1), synth.Scene(64, 1, 16, 5, 1))
    w = synth.Workload("gated", base.n_q_heads, base.n_kv_heads, base.head_dim, 1024, "bf16", "peaked", 0.9, 1.0,
                       scenes, page_tokens=64, seed=23)
    ctx = harness.create_context(w)
    try:
        gs, refs, qs, ks, vs = [], [], [], [], []
        for i, sc in enumerate(scenes):
            gs.append(harness.GpuScene(ctx, w, i))
            pk, pv = synth.make_prefix(w, i)
            q, k, v = synth.make_qkv(w, i, 0, 0, 0)
            empty = ([np.zeros((0, w.n_kv_heads, w.head_dim), dtype=np.uint16)] * sc.n_forks,) * 2
            refs.append(pu.attention_oracle(w, (pk, pv), empty, q, k, v))
            qs.append(q); ks.append(k); vs.append(v)
        pack = lambda xs: harness.bf16_tensor(np.concatenate([x.reshape(-1) for x in xs]))
        qd, kd, vd = pack(qs), pack(ks), pack(vs)
        n_total = sum(sc.n_forks for sc in scenes)
        rng = np.random.default_rng(5)
        some = rng.integers(0, 3, n_total).astype(np.int32) * 7          # about a third are 0
        some[5:7] = 0                                                    # scene 1 sits out as a whole
        gates = [some, np.ones(n_total, np.int32), np.zeros(n_total, np.int32),
                 (np.arange(n_total) == 11).astype(np.int32)]
        for gate in gates:
            out = torch.full_like(qd, float("nan"))
            n0 = fdd.fdd_launch_count(ctx)
            fdd.fdd_block_attn_gated(ctx, [g.forkset for g in gs], 0, qd, kd, vd, out,
                                     [sc.block_len for sc in scenes], 1.0 / np.sqrt(w.head_dim), 0,
                                     torch.from_numpy(gate).cuda())
            fdd.fdd_poll_status(ctx)
            assert fdd.fdd_launch_count(ctx) - n0 == 1
            got = out.float().cpu().numpy().astype(np.float64)
            off = fork = 0
            for sc, ref in zip(scenes, refs):
                rows = got[off:off + ref.size].reshape(ref.shape)
                for f in range(sc.n_forks):
                    if gate[fork + f]:
                        pu.assert_attention_close(rows[f], ref[f])
                    else:
                        assert np.all(np.isnan(rows[f])), "a skipped rollout was written"
                off += ref.size; fork += sc.n_forks
    finally:
        fdd.fdd_destroy(ctx)
    # the CUDA-core kernel (GQA group of three) honours the gate as well
    w = synth.Workload("g3_gated", 6, 2, 64, 256, "f32", "peaked", 0.9, 0.0,
                       (synth.Scene(prefix_len=100, n_forks=3, block_len=16, n_scaffold=5, n_blocks=1),), seed=13)
    ctx = harness.create_context(w)
    try:
        g = harness.GpuScene(ctx, w, 0)
        pk, pv = synth.make_prefix(w, 0)
        q, k, v = synth.make_qkv(w, 0, 0, 0, 0)
        empty = ([np.zeros((0, w.n_kv_heads, w.head_dim), dtype=np.uint16)] * 3,) * 2
        ref = pu.attention_oracle(w, (pk, pv), empty, q, k, v)
        out = torch.full((q.size,), float("nan"), dtype=torch.bfloat16, device="cuda")
        fdd.fdd_block_attn_gated(ctx, [g.forkset], 0, harness.bf16_tensor(q), harness.bf16_tensor(k),
                                 harness.bf16_tensor(v), out, [16], 1.0 / np.sqrt(w.head_dim), 0,
                                 torch.tensor([4, 0, 1], dtype=torch.int32, device="cuda"))
        fdd.fdd_poll_status(ctx)
        got = out.float().cpu().numpy().astype(np.float64).reshape(ref.shape)
        pu.assert_attention_close(got[[0, 2]], ref[[0, 2]])
        assert np.all(np.isnan(got[1]))
    finally:
        fdd.fdd_destroy(ctx)


def test_attention_repeated_calls_reuse_scratch():
    # the scratch of the split-unit merge is reusable at once: the same call three times in a row
    # (different inputs) stays correct
    w = synth.workload("tts")
    ctx = harness.create_context(w)
    try:
        scene = harness.GpuScene(ctx, w, 0)
        pk, pv = synth.make_prefix(w, 0)
        empty = ([np.zeros((0, w.n_kv_heads, w.head_dim), dtype=np.uint16)] * 8,) * 2
        for step in range(3):
            q, k, v = synth.make_qkv(w, 0, 0, 0, step)
            got = pu.attention_gpu(ctx, scene, q, k, v)
            ref = pu.attention_oracle(w, (pk, pv), empty, q, k, v, forks=[step, 7 - step])
            pu.assert_attention_close(got[[step, 7 - step]], ref)
    finally:
        fdd.fdd_destroy(ctx)


def test_serving_mix_full_size_one_call():
    # the ragged serving batch at full size: 16 scenes (prefix 2048..12288 tokens in shuffled pages,
    # 1/4/16 rollouts, blocks of 16/32/64) in ONE attention call and ONE unmask call; the oracle
    # checks one rollout of every third scene (attention) and of three scenes (unmask)
    w = synth.workload("serving_mix")
    ctx = harness.create_context(w)
    try:
        scenes = w.scenes
        gs = [harness.GpuScene(ctx, w, i) for i in range(len(scenes))]
        qs, ks, vs = zip(*[synth.make_qkv(w, i, 0, 0, 0) for i in range(len(scenes))])
        pack = lambda xs: harness.bf16_tensor(np.concatenate([x.reshape(-1) for x in xs]))
        qd, kd, vd = pack(qs), pack(ks), pack(vs)
        out = torch.full_like(qd, float("nan"))
        n0 = fdd.fdd_launch_count(ctx)
        fdd.fdd_block_attn(ctx, [g.forkset for g in gs], 0, qd, kd, vd, out, [sc.block_len for sc in scenes],
                           1.0 / np.sqrt(w.head_dim), 0)
        fdd.fdd_poll_status(ctx)
        assert fdd.fdd_launch_count(ctx) - n0 == 1
        got = out.float().cpu().numpy().astype(np.float64)
        assert np.all(np.isfinite(got))
        off = 0
        for i, sc in enumerate(scenes):
            n = qs[i].size
            if i % 3 == 0:
                f = (i * 5) % sc.n_forks
                pk, pv = synth.make_prefix(w, i)
                empty = ([np.zeros((0, w.n_kv_heads, w.head_dim), dtype=np.uint16)] * sc.n_forks,) * 2
                ref = pu.attention_oracle(w, (pk, pv), empty, qs[i], ks[i], vs[i], forks=[f])
                pu.assert_attention_close(got[off:off + n].reshape(qs[i].shape)[[f]], ref)
            off += n
        # unmask: all 16 scenes in one call; logits rows are generated for the checked rollouts only
        # (the other rollouts of a checked scene reuse them, unchecked scenes get one shared row)
        checked = {2: 0, 7: None, 11: None}
        for i in (7, 11):
            checked[i] = scenes[i].n_forks - 1
        toks, sts, lgs = [], [], []
        shared_row = synth.make_logits_row(w, 0, 0, 0, 0, 0)
        for i, sc in enumerate(scenes):
            t_, s_ = synth.make_block_template(w, i, 0)
            lg = np.empty((sc.n_forks, sc.block_len, w.vocab), dtype=np.uint16)
            lg[:] = shared_row
            if i in checked:
                frozen = set(synth.scaffold_positions(w, i, 0).tolist())
                for pos in range(sc.block_len):
                    if pos not in frozen:
                        lg[:, pos] = synth.make_logits_row(w, i, 0, 0, checked[i], pos)
            toks.append(t_); sts.append(s_); lgs.append(lg)
        lg_d = harness.bf16_tensor(np.concatenate([x.reshape(-1) for x in lgs]))
        tok_d = torch.from_numpy(np.concatenate([x.reshape(-1) for x in toks])).cuda()
        st_d = torch.from_numpy(np.concatenate([x.reshape(-1) for x in sts])).cuda()
        total_forks = sum(sc.n_forks for sc in scenes)
        n_comm = torch.full((total_forks,), -7, dtype=torch.int32, device="cuda")
        n_left = torch.full((total_forks,), -7, dtype=torch.int32, device="cuda")
        conf = torch.zeros(tok_d.shape, dtype=torch.float32, device="cuda")
        n0 = fdd.fdd_launch_count(ctx)
        fdd.fdd_unmask(ctx, [g.forkset for g in gs], lg_d, tok_d, st_d, [sc.block_len for sc in scenes],
                       w.threshold, w.temperature, 0, 0, n_comm, n_left, conf)
        fdd.fdd_poll_status(ctx)
        assert fdd.fdd_launch_count(ctx) - n0 == 3        # all scenes in one pair of launches, after one that stores the 151 seeds
        tok_h, st_h, conf_h = tok_d.cpu().numpy(), st_d.cpu().numpy(), conf.cpu().numpy()
        nc_h, nl_h = n_comm.cpu().numpy(), n_left.cpu().numpy()
        assert np.all(nc_h >= 1) and np.all(nl_h >= 0)
        row_off = fork_off = 0
        ambiguous = 0
        for i, sc in enumerate(scenes):
            rows = sc.n_forks * sc.block_len
            if i in checked:
                f = checked[i]
                sl = slice(row_off + f * sc.block_len, row_off + (f + 1) * sc.block_len)
                ref = unmask_step(pu.widen_logits(w, lgs[i][[f]]), toks[i][[f]], sts[i][[f]], gs[i].seeds[[f]],
                                  w.threshold, w.temperature, 0, 0)
                sub = dict(tokens=tok_h[sl][None], state=st_h[sl][None], conf=conf_h[sl][None],
                           n_committed=nc_h[fork_off + f:fork_off + f + 1], n_left=nl_h[fork_off + f:fork_off + f + 1])
                info = pu.compare_unmask(sub, ref, toks[i][[f]], sts[i][[f]], w.threshold)
                ambiguous += len(info["ambiguous_forks"])
            row_off += rows
            fork_off += sc.n_forks
        assert ambiguous <= 1
    finally:
        fdd.fdd_destroy(ctx)


def test_attention_largest_block_and_group():
    # the limits of the interface: block of 128 positions, 16 query heads per KV head (2048 stacked
    # rows per rollout and KV head = 8 row pairs), head_dim 64, with an earlier block in the suffix
    sc = synth.Scene(prefix_len=389, n_forks=2, block_len=128, n_scaffold=30, n_blocks=2)
    w = synth.Workload("wide", 16, 1, 64, 512, "bf16", "peaked", 0.9, 1.0, (sc,), qkv_sigma=0.5, seed=31)
    ctx = harness.create_context(w)
    try:
        scene = harness.GpuScene(ctx, w, 0, suffix_capacity=256)
        pk, pv = synth.make_prefix(w, 0)
        ofs = ForkSet([pk], [pv], 2, scene.seeds)
        _, kb, vb = synth.make_qkv(w, 0, 0, 0, 0)
        fdd.fdd_kv_commit(ctx, [scene.forkset], 0, harness.bf16_tensor(kb), harness.bf16_tensor(vb), [128], 1)
        ofs.kv_commit(0, kb, vb)
        q, k, v = synth.make_qkv(w, 0, 0, 1, 0)
        for causal in (False, True):
            got = pu.attention_gpu(ctx, scene, q, k, v, causal=causal)
            ref = pu.attention_oracle(w, (pk, pv), _suffix_from_oracle(ofs), q, k, v, causal=causal)
            pu.assert_attention_close(got, ref)
    finally:
        fdd.fdd_destroy(ctx)


def test_attention_group_of_three_uses_the_cuda_core_kernel():
    # a GQA group that is not a power of two is outside the tensor-core kernel's row stacking
    sc = synth.Scene(prefix_len=150, n_forks=2, block_len=20, n_scaffold=5, n_blocks=1)
    w = synth.Workload("g3", 6, 2, 64, 512, "bf16", "peaked", 0.9, 1.0, (sc,), qkv_sigma=0.5, seed=32)
    _attention_case(w)


def test_more_scenes_and_rows_than_one_launch_takes():
    # 18 scenes (more than the 16 of one attention / unmask launch) and, separately, three sets of
    # 4096 rows each (more than the 8192 rows of one unmask launch): the calls split the work
    scenes = tuple(synth.Scene(prefix_len=70 + 13 * i, n_forks=1 + i % 3, block_len=16, n_scaffold=4, n_blocks=1)
                   for i in range(18))
    w = synth.Workload("many", 8, 2, 64, 640, "bf16", "peaked", 0.9, 0.7, scenes, qkv_sigma=0.5, seed=41)
    ctx = harness.create_context(w)
    try:
        gs = [harness.GpuScene(ctx, w, i) for i in range(len(scenes))]
        qs, ks, vs = zip(*[synth.make_qkv(w, i, 0, 0, 0) for i in range(len(scenes))])
        pack = lambda xs: harness.bf16_tensor(np.concatenate([x.reshape(-1) for x in xs]))
        qd, kd, vd = pack(qs), pack(ks), pack(vs)
        out = torch.full_like(qd, float("nan"))
        n0 = fdd.fdd_launch_count(ctx)
        fdd.fdd_block_attn(ctx, [g.forkset for g in gs], 0, qd, kd, vd, out, [16] * 18, 0.125, 0)
        fdd.fdd_poll_status(ctx)
        assert fdd.fdd_launch_count(ctx) - n0 == 2
        got = out.float().cpu().numpy().astype(np.float64)
        off = 0
        for i, sc in enumerate(scenes):
            pk, pv = synth.make_prefix(w, i)
            empty = ([np.zeros((0, w.n_kv_heads, w.head_dim), dtype=np.uint16)] * sc.n_forks,) * 2
            ref = pu.attention_oracle(w, (pk, pv), empty, qs[i], ks[i], vs[i], scale=0.125)
            pu.assert_attention_close(got[off:off + ref.size].reshape(ref.shape), ref)
            off += ref.size
        toks, sts, lgs = zip(*[synth.make_block_template(w, i, 0) + (synth.make_logits(w, i, 0, 0, rows="all"),)
                               for i in range(len(scenes))])
        flat = lambda xs: np.concatenate([x.reshape(-1) for x in xs])
        tok_d, st_d = torch.from_numpy(flat(toks)).cuda(), torch.from_numpy(flat(sts)).cuda()
        nf = sum(sc.n_forks for sc in scenes)
        n_c = torch.zeros(nf, dtype=torch.int32, device="cuda"); n_l = torch.zeros(nf, dtype=torch.int32, device="cuda")
        n0 = fdd.fdd_launch_count(ctx)
        fdd.fdd_unmask(ctx, [g.forkset for g in gs], harness.bf16_tensor(flat(lgs)), tok_d, st_d, [16] * 18,
                       w.threshold, w.temperature, 0, 0, n_c, n_l)
        fdd.fdd_poll_status(ctx)
        assert fdd.fdd_launch_count(ctx) - n0 == 5                 # the seeds of all 18 scenes, then 16 scenes, then 2
        tok_h, st_h = tok_d.cpu().numpy(), st_d.cpu().numpy()
        off = foff = 0
        for i, sc in enumerate(scenes):
            rows = sc.n_forks * 16
            ref = unmask_step(pu.widen_logits(w, lgs[i]), toks[i], sts[i], gs[i].seeds, w.threshold, w.temperature, 0, 0)
            sub = dict(tokens=tok_h[off:off + rows].reshape(sc.n_forks, 16), state=st_h[off:off + rows].reshape(sc.n_forks, 16),
                       conf=None, n_committed=n_c.cpu().numpy()[foff:foff + sc.n_forks], n_left=n_l.cpu().numpy()[foff:foff + sc.n_forks])
            assert len(pu.compare_unmask(sub, ref, toks[i], sts[i], w.threshold)["ambiguous_forks"]) <= 1
            off += rows; foff += sc.n_forks
    finally:
        fdd.fdd_destroy(ctx)
    # rows: 3 sets x (32 rollouts x 128 positions) = 12288 rows > 8192 per launch
    big = tuple(synth.Scene(prefix_len=16, n_forks=32, block_len=128, n_scaffold=40, n_blocks=1) for _ in range(3))
    w = synth.Workload("rows", 4, 1, 64, 512, "f32", "peaked", 0.6, 1.1, big, seed=42)
    ctx = harness.create_context(w)
    try:
        gs = [harness.GpuScene(ctx, w, i) for i in range(3)]
        toks, sts, lgs = zip(*[synth.make_block_template(w, i, 0) + (synth.make_logits(w, i, 0, 0, rows="all"),)
                               for i in range(3)])
        flat = lambda xs: np.concatenate([x.reshape(-1) for x in xs])
        tok_d, st_d = torch.from_numpy(flat(toks)).cuda(), torch.from_numpy(flat(sts)).cuda()
        n_c = torch.zeros(96, dtype=torch.int32, device="cuda"); n_l = torch.zeros(96, dtype=torch.int32, device="cuda")
        n0 = fdd.fdd_launch_count(ctx)
        fdd.fdd_unmask(ctx, [g.forkset for g in gs], torch.from_numpy(flat(lgs)).cuda(), tok_d, st_d, [128] * 3,
                       w.threshold, w.temperature, 0, 0, n_c, n_l)
        fdd.fdd_poll_status(ctx)
        assert fdd.fdd_launch_count(ctx) - n0 == 5                 # the seeds, two sets, then one
        tok_h, st_h = tok_d.cpu().numpy().reshape(3, 32, 128), st_d.cpu().numpy().reshape(3, 32, 128)
        amb = 0
        for i in (0, 2):
            f = [3, 30]
            ref = unmask_step(lgs[i][f].astype(np.float64), toks[i][f], sts[i][f], gs[i].seeds[f], w.threshold,
                              w.temperature, 0, 0)
            sub = dict(tokens=tok_h[i][f], state=st_h[i][f], conf=None,
                       n_committed=n_c.cpu().numpy().reshape(3, 32)[i][f], n_left=n_l.cpu().numpy().reshape(3, 32)[i][f])
            amb += len(pu.compare_unmask(sub, ref, toks[i][f], sts[i][f], w.threshold)["ambiguous_forks"])
        assert amb <= 1
    finally:
        fdd.fdd_destroy(ctx)


def test_unmask_counted_matches_unmask_with_the_step_passed_by_value():
    # 18 scenes (two groups of launches inside one call): the device-side step counter must advance
    # once per call, not once per group, and give the same draws as the step passed by value
    scenes = tuple(synth.Scene(prefix_len=40, n_forks=1 + i % 2, block_len=16, n_scaffold=4, n_blocks=1) for i in range(18))
    w = synth.Workload("counted", 8, 2, 64, 512, "f32", "peaked", 0.95, 0.8, scenes, seed=77)
    ctx = harness.create_context(w)
    try:
        gs = [harness.GpuScene(ctx, w, i) for i in range(18)]
        sets = [g.forkset for g in gs]
        flat = lambda xs: np.concatenate([x.reshape(-1) for x in xs])
        toks, sts = zip(*[synth.make_block_template(w, i, 0) for i in range(18)])
        nf = sum(sc.n_forks for sc in scenes)
        results = []
        for counted in (False, True):
            tok_d, st_d = torch.from_numpy(flat(toks)).cuda(), torch.from_numpy(flat(sts)).cuda()
            n_c = torch.zeros(nf, dtype=torch.int32, device="cuda"); n_l = torch.zeros(nf, dtype=torch.int32, device="cuda")
            counter = torch.zeros(1, dtype=torch.int32, device="cuda")
            trace = []
            for step in range(3):
                lg = torch.from_numpy(flat([synth.make_logits(w, i, 0, step, rows="all") for i in range(18)])).cuda()
                if counted:
                    fdd.fdd_unmask_counted(ctx, sets, lg, tok_d, st_d, [16] * 18, w.threshold, w.temperature, 0, counter, n_c, n_l)
                else:
                    fdd.fdd_unmask(ctx, sets, lg, tok_d, st_d, [16] * 18, w.threshold, w.temperature, 0, step, n_c, n_l)
                trace.append((tok_d.cpu().numpy(), st_d.cpu().numpy(), n_c.cpu().numpy(), n_l.cpu().numpy()))
            fdd.fdd_poll_status(ctx)
            if counted:
                assert int(counter.item()) == 3
            results.append(trace)
        for a_, b_ in zip(*results):
            for x, y in zip(a_, b_):
                assert np.array_equal(x, y)
        assert results[0][0][2].sum() > 0 and not np.array_equal(results[0][0][0], results[0][2][0])
    finally:
        fdd.fdd_destroy(ctx)


def test_prefix_is_never_written_and_forks_with_equal_inputs_agree():
    w = synth.small_variant(synth.workload("tts"), prefix_len=512, vocab=512, n_forks=4, n_blocks=1)
    ctx = harness.create_context(w)
    try:
        scene = harness.GpuScene(ctx, w, 0)
        before = [t.clone() for t in scene.prefix_k + scene.prefix_v]
        q, k, v = synth.make_qkv(w, 0, 0, 0, 0)
        q, k, v = (np.repeat(x[:1], 4, axis=0) for x in (q, k, v))
        got = pu.attention_gpu(ctx, scene, q, k, v)
        # Rollouts with equal inputs agree up to the rounding of the bf16 output: a unit may be cut
        # between CTAs at a different key tile per rollout, which changes the summation order only.
        for f in range(1, 4):
            assert np.max(np.abs(got[f] - got[0])) <= 2e-3
            assert np.linalg.norm(got[f] - got[0]) <= 4e-3 * np.linalg.norm(got[0])
        fdd.fdd_kv_commit(ctx, [scene.forkset], 0, harness.bf16_tensor(k), harness.bf16_tensor(v), [k.shape[1]], 1)
        fdd.fdd_poll_status(ctx)
        for a, b in zip(before, scene.prefix_k + scene.prefix_v):
            assert torch.equal(a, b)
    finally:
        fdd.fdd_destroy(ctx)


# ---------------------------------------------------------------------------------------------
# kv commit
# ---------------------------------------------------------------------------------------------
def test_kv_commit_bytes_and_capacity():
    w = synth.small_variant(synth.workload("tts"), prefix_len=64, vocab=512, n_forks=3, n_blocks=2)
    ctx = harness.create_context(w)
    try:
        scene = harness.GpuScene(ctx, w, 0, suffix_capacity=2 * w.scenes[0].block_len)
        d = w.scenes[0].block_len
        blocks = [synth.make_qkv(w, 0, 0, b, 0)[1:] for b in range(2)]
        for b, (kb, vb) in enumerate(blocks):
            fdd.fdd_kv_commit(ctx, [scene.forkset], 0, harness.bf16_tensor(kb), harness.bf16_tensor(vb), [d], 1)
        fdd.fdd_poll_status(ctx)
        sk = scene.suffix_k[0].view(torch.int16).cpu().numpy().view(np.uint16)    # [N,Hkv,cap,D]
        sv = scene.suffix_v[0].view(torch.int16).cpu().numpy().view(np.uint16)
        for b, (kb, vb) in enumerate(blocks):
            assert np.array_equal(sk[:, :, b * d:(b + 1) * d], kb.transpose(0, 2, 1, 3))
            assert np.array_equal(sv[:, :, b * d:(b + 1) * d], vb.transpose(0, 2, 1, 3))
        with pytest.raises(fdd.FddError) as ei:
            fdd.fdd_kv_commit(ctx, [scene.forkset], 0, harness.bf16_tensor(blocks[0][0]),
                              harness.bf16_tensor(blocks[0][1]), [d], 1)
        assert ei.value.status == fdd.FDD_ERR_CAPACITY
        fdd.fdd_forkset_reset(ctx, scene.forkset)
        assert fdd.fdd_forkset_suffix_len(scene.forkset) == 0
    finally:
        fdd.fdd_destroy(ctx)


# ---------------------------------------------------------------------------------------------
# unmask
# ---------------------------------------------------------------------------------------------
def _unmask_step_case(w, block=0, step=0, threshold=None, temperature=None, state_override=None):
    ctx = harness.create_context(w)
    try:
        scene = harness.GpuScene(ctx, w, 0)
        tokens, state = synth.make_block_template(w, 0, block)
        if state_override is not None:
            tokens, state = state_override(tokens, state)
        logits = synth.make_logits(w, 0, block, step, rows="all")
        th = w.threshold if threshold is None else threshold
        te = w.temperature if temperature is None else temperature
        got = pu.unmask_gpu(ctx, scene, logits, tokens, state, th, te, block, step)
        ref = unmask_step(pu.widen_logits(w, logits), tokens, state, scene.seeds, th, te, block, step)
        return pu.compare_unmask(got, ref, tokens, state, th), got, ref
    finally:
        fdd.fdd_destroy(ctx)


def test_unmask_tiny_fallback_every_step():
    w = synth.workload("tiny")
    ctx = harness.create_context(w)
    try:
        scene = harness.GpuScene(ctx, w, 0)
        tokens, state = synth.make_block_template(w, 0, 0)
        steps = 0
        while np.any(state == MASKED):
            logits = synth.make_logits(w, 0, 0, steps, rows="all")
            got = pu.unmask_gpu(ctx, scene, logits, tokens, state, w.threshold, 0.0, 0, steps)
            ref = unmask_step(logits, tokens, state, scene.seeds, w.threshold, 0.0, 0, steps)
            info = pu.compare_unmask(got, ref, tokens, state, w.threshold)
            assert not info["ambiguous_forks"]
            assert got["n_committed"][0] == 1
            tokens, state = got["tokens"], got["state"]
            steps += 1
            assert steps <= 16
        assert steps == 12
    finally:
        fdd.fdd_destroy(ctx)


@pytest.mark.parametrize("temperature", [0.0, 1.0])
def test_unmask_full_vocab_bf16(temperature):
    w = synth.small_variant(synth.workload("tts"), prefix_len=64, n_forks=4, n_blocks=1)
    info, got, ref = _unmask_step_case(w, temperature=temperature)
    assert info["rows"] == 4 * 22
    assert len(info["ambiguous_forks"]) <= 1
    assert got["n_committed"].sum() >= 4


def test_unmask_odd_vocab_and_partial_state():
    # vocabulary not a multiple of the vector width, several chunks with a ragged tail, rows in
    # every state, one rollout already finished
    sc = synth.Scene(prefix_len=16, n_forks=3, block_len=9, n_scaffold=2, n_blocks=1)
    w = synth.Workload("odd", 4, 1, 64, 8192 * 2 + 1237, "f32", "peaked", 0.7, 0.8, (sc,), seed=21)

    def override(tokens, state):
        state = state.copy()
        tokens = tokens.copy()
        state[1][state[1] == MASKED] = COMMITTED          # rollout 1 is done
        tokens[1] = 5
        first = np.nonzero(state[2] == MASKED)[0][0]
        state[2, first] = COMMITTED
        tokens[2, first] = 77
        return tokens, state

    info, got, ref = _unmask_step_case(w, state_override=override)
    assert got["n_committed"][1] == 0 and got["n_left"][1] == 0
    assert not info["ambiguous_forks"]
    w2 = synth.Workload("odd_bf16", 4, 1, 64, 8192 + 3, "bf16", "peaked", 0.7, 1.3, (sc,), seed=22)
    info, _, _ = _unmask_step_case(w2)
    assert not info["ambiguous_forks"]


@pytest.mark.parametrize("recipe,dtype,vocab,temperature", [
    ("normal_sigma2", "bf16", 151936, 1.0),
    ("normal_sigma2", "bf16", 151936, 0.05),
    ("normal_sigma2", "bf16", 151936, 2.0),
    ("normal_sigma2", "f32", 8192 * 2 + 1237, 1.0),      # rows that bulk copies cannot address
    ("normal_sigma2", "f32", 50000, 0.05),
    ("constant", "bf16", 151936, 1.0),
    ("constant", "f32", 4099, 0.7),
])
def test_unmask_noise_decides_on_flat_and_equal_rows(recipe, dtype, vocab, temperature):
    # The hard case of the sampled trajectory section: no id towers over the rest, so the noise
    # decides the arg-max and the pruning of the kernel has to keep every id that can still win.
    # Threshold below any probability: every MASKED row commits, and every row's token is compared.
    sc = synth.Scene(prefix_len=16, n_forks=2, block_len=8, n_scaffold=2, n_blocks=1)
    w = synth.Workload("flat", 4, 1, 64, vocab, dtype, recipe, -1.0, temperature, (sc,), seed=31)
    for step in (0, 3):
        info, got, ref = _unmask_step_case(w, step=step)
        assert info["rows"] == 2 * 6 and not info["ambiguous_forks"] or info["low_margin_rows"] > 0
        masked = ref["choice"] >= 0
        clear = masked & (ref["score_margin"] > pu.SCORE_MARGIN)
        assert clear.sum() >= 2 * 6 - 2
        assert np.array_equal(got["tokens"][clear], ref["choice"][clear])
        assert np.all(got["state"][masked] == COMMITTED)
        if recipe == "constant":
            assert len(set(got["tokens"][masked].tolist())) >= 8        # the winners are spread over the vocabulary


def test_unmask_threshold_extremes():
    w = synth.small_variant(synth.workload("tts"), prefix_len=64, vocab=4096, n_forks=2, n_blocks=1)
    info, got, ref = _unmask_step_case(w, threshold=1.5)          # nothing passes: one commit each
    assert list(got["n_committed"]) == [1, 1]
    info, got, ref = _unmask_step_case(w, threshold=-1.0)         # everything commits
    assert np.all(got["state"] != MASKED) and list(got["n_left"]) == [0, 0]


def test_unmask_identical_seeds_give_identical_forks():
    w = synth.small_variant(synth.workload("tts"), prefix_len=64, vocab=4096, n_forks=3, n_blocks=1)
    ctx = harness.create_context(w)
    try:
        scene = harness.GpuScene(ctx, w, 0, identical_seeds=True)
        tokens, state = synth.make_block_template(w, 0, 0)
        logits = np.repeat(synth.make_logits(w, 0, 0, 0, rows="all")[:1], 3, axis=0)
        got = pu.unmask_gpu(ctx, scene, logits, tokens, state, w.threshold, 1.0, 0, 0)
        for f in (1, 2):
            assert np.array_equal(got["tokens"][f], got["tokens"][0])
            assert np.array_equal(got["state"][f], got["state"][0])
    finally:
        fdd.fdd_destroy(ctx)


def test_unmask_long_prefix_full_size_step0():
    # the largest configuration at full size: all 2048 rows on the GPU; the oracle checks every
    # row of four sampled rollouts (1216 vocabulary-wide rows would take minutes on the CPU)
    w = synth.workload("long_prefix")
    ctx = harness.create_context(w)
    try:
        scene = harness.GpuScene(ctx, w, 0)
        tokens, state = synth.make_block_template(w, 0, 0)
        sample = [0, 7, 19, 31]
        logits = np.zeros((32, 64, w.vocab), dtype=np.uint16)
        frozen = set(synth.scaffold_positions(w, 0, 0).tolist())
        for f in sample:
            for i in range(64):
                if i not in frozen:
                    logits[f, i] = synth.make_logits_row(w, 0, 0, 0, f, i)
        for f in range(32):      # rollouts outside the sample reuse rollout 0's rows (less host time)
            if f not in sample:
                logits[f] = logits[0]
        got = pu.unmask_gpu(ctx, scene, logits, tokens, state, w.threshold, w.temperature, 0, 0)
        ref = unmask_step(pu.widen_logits(w, logits[sample]), tokens[sample], state[sample],
                          scene.seeds[sample], w.threshold, w.temperature, 0, 0)
        sub = {k: (v[sample] if v is not None else None) for k, v in got.items()}
        info = pu.compare_unmask(sub, ref, tokens[sample], state[sample], w.threshold)
        assert info["rows"] == 4 * 38
        assert len(info["ambiguous_forks"]) <= 1
        assert np.all(got["n_committed"] >= 1)
        assert np.all(got["n_left"] + got["n_committed"] == 38)
    finally:
        fdd.fdd_destroy(ctx)


# ---------------------------------------------------------------------------------------------
# Scaffold Speculative Decoding: draft and accept scan
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("temperature", [0.0, 0.9])
def test_ss_draft_and_accept_cycles_match_oracle(temperature):
    from oracle.ss import DRAFT, ss_accept, ss_draft
    w = synth.small_variant(synth.workload("tts"), prefix_len=64, vocab=8192 + 4096, n_forks=5, n_blocks=1)
    sc = w.scenes[0]
    ctx = harness.create_context(w)
    try:
        scene = harness.GpuScene(ctx, w, 0)
        tokens, state = synth.make_block_template(w, 0, 0)
        n_a = torch.full((sc.n_forks,), -7, dtype=torch.int32, device="cuda")
        n_l = torch.full((sc.n_forks,), -7, dtype=torch.int32, device="cuda")
        g = np.random.default_rng(77)
        cycle = 0
        while np.any(state == MASKED):
            # draft
            logits = synth.make_logits(w, 0, 0, cycle, rows="all")
            tok_d, st_d = torch.from_numpy(tokens).cuda(), torch.from_numpy(state).cuda()
            fdd.fdd_ss_draft(ctx, [scene.forkset], harness.logits_tensor(w, logits), tok_d, st_d, [sc.block_len],
                             temperature, 0, 2 * cycle, n_a, n_l)
            fdd.fdd_poll_status(ctx)
            ref_t, ref_s = ss_draft(pu.widen_logits(w, logits), tokens, state, scene.seeds, temperature, 0, 2 * cycle)
            margins = unmask_step(pu.widen_logits(w, logits), tokens, state, scene.seeds, -1.0, temperature, 0,
                                  2 * cycle)["score_margin"]
            got_t, got_s = tok_d.cpu().numpy(), st_d.cpu().numpy()
            assert np.array_equal(got_s, ref_s) and not np.any(got_s == MASKED)
            clear = margins > pu.SCORE_MARGIN
            assert np.array_equal(got_t[clear], ref_t[clear]) and clear.mean() > 0.99
            assert np.array_equal(n_a.cpu().numpy(), (state == MASKED).sum(axis=1)) and not n_l.cpu().numpy().any()
            tokens, state = ref_t, ref_s                    # continue from the oracle's drafts
            # verifier logits: agrees with the first k_f drafts of rollout f, then with nothing in particular
            ar = (g.standard_normal((sc.n_forks, sc.block_len, w.vocab)) * 0.5).astype(np.float32)
            for f in range(sc.n_forks):
                drafts = np.nonzero(state[f] == DRAFT)[0]
                k = int(g.integers(0, len(drafts) + 1)) if f else len(drafts)      # rollout 0: all accepted
                for i in drafts[:k]:
                    ar[f, i, tokens[f, i]] = 12.0
            ar_bits = synth.f32_to_bf16_bits(ar)
            tok_d, st_d = torch.from_numpy(tokens).cuda(), torch.from_numpy(state).cuda()
            fdd.fdd_ss_accept(ctx, [scene.forkset], harness.bf16_tensor(ar_bits), tok_d, st_d, [sc.block_len],
                              temperature, 0, 2 * cycle + 1, n_a, n_l)
            fdd.fdd_poll_status(ctx)
            ref = ss_accept(pu.widen_logits(w, ar_bits), tokens, state, scene.seeds, temperature, 0, 2 * cycle + 1)
            got_t, got_s = tok_d.cpu().numpy(), st_d.cpu().numpy()
            for f in range(sc.n_forks):
                if np.all(ref["score_margin"][f] > pu.SCORE_MARGIN):
                    assert np.array_equal(got_t[f], ref["tokens"][f]) and np.array_equal(got_s[f], ref["state"][f])
                    assert n_a.cpu().numpy()[f] == ref["n_accepted"][f] and n_l.cpu().numpy()[f] == ref["n_left"][f]
            keep = state == SCAFFOLD
            assert np.array_equal(got_t[keep], tokens[keep]) and np.all(got_s[keep] == SCAFFOLD)
            assert not np.any(got_s == DRAFT)
            tokens, state = ref["tokens"], ref["state"]
            cycle += 1
            assert cycle <= sc.block_len
        assert cycle >= 2
    finally:
        fdd.fdd_destroy(ctx)


# ---------------------------------------------------------------------------------------------
# whole block loop, averaging
# ---------------------------------------------------------------------------------------------
def test_block_loop_matches_oracle_and_averages():
    w = synth.small_variant(synth.workload("tts"), prefix_len=200, vocab=2048, n_forks=4, n_blocks=2)
    sc = w.scenes[0]
    ctx = harness.create_context(w)
    try:
        scene = harness.GpuScene(ctx, w, 0)
        pk, pv = synth.make_prefix(w, 0)
        ofs = ForkSet([pk], [pv], sc.n_forks, scene.seeds)
        scale = 1.0 / np.sqrt(w.head_dim)
        all_tokens, all_state = [], []
        diverged = set()
        for block in range(sc.n_blocks):
            tokens, state = synth.make_block_template(w, 0, block)
            step = 0
            while np.any(state == MASKED):
                q, k, v = synth.make_qkv(w, 0, 0, block, step)
                got_attn = pu.attention_gpu(ctx, scene, q, k, v)
                ref_attn = pu.attention_oracle(w, (pk, pv), _suffix_from_oracle(ofs), q, k, v)
                pu.assert_attention_close(got_attn, ref_attn)
                logits = synth.make_logits(w, 0, block, step, rows="all")
                got = pu.unmask_gpu(ctx, scene, logits, tokens, state, w.threshold, w.temperature, block, step)
                ref = unmask_step(pu.widen_logits(w, logits), tokens, state, scene.seeds, w.threshold,
                                  w.temperature, block, step)
                info = pu.compare_unmask(got, ref, tokens, state, w.threshold)
                diverged |= info["ambiguous_forks"]
                tokens, state = got["tokens"], got["state"]
                step += 1
                assert step <= sc.block_len
            fdd.fdd_kv_commit(ctx, [scene.forkset], 0, harness.bf16_tensor(k), harness.bf16_tensor(v), [sc.block_len], 1)
            ofs.kv_commit(0, k, v)
            all_tokens.append(tokens)
            all_state.append(state)
        assert len(diverged) <= 1
        toks, sts = np.concatenate(all_tokens, axis=1), np.concatenate(all_state, axis=1)
        traj = synth.tokens_to_trajectory(w, toks, sts)
        t_dev = torch.from_numpy(traj).cuda()
        out = torch.zeros((w.waypoints, 2), dtype=torch.float32, device="cuda")
        fdd.fdd_average_rollouts(ctx, t_dev, sc.n_forks, w.waypoints, out)
        fdd.fdd_poll_status(ctx)
        ref = average_rollouts(traj)
        got = out.cpu().numpy().astype(np.float64)
        assert np.all(np.abs(got - ref) <= 1e-5 * np.maximum(np.abs(ref), 1e-30) + 1e-30)
    finally:
        fdd.fdd_destroy(ctx)


def test_pipelined_block_loop_gated_attention_one_step_ahead():
    # The loop as a server runs it: everything stays on the device, attention is gated by the
    # n_left array of the step before, and step t + 1 is enqueued before the host has read the
    # counts of step t.  Every step is recorded on the device and re-done by the oracle afterwards:
    # rollouts that still decode get the oracle's attention, finished ones are never written, the
    # step enqueued after the block was complete does nothing at all.
    w = synth.small_variant(synth.workload("tts"), prefix_len=300, vocab=2048, n_forks=6)
    sc = w.scenes[0]
    N, d = sc.n_forks, sc.block_len
    ctx = harness.create_context(w)
    try:
        scene = harness.GpuScene(ctx, w, 0)
        pk, pv = synth.make_prefix(w, 0)
        empty = ([np.zeros((0, w.n_kv_heads, w.head_dim), dtype=np.uint16)] * N,) * 2
        tokens0, state0 = synth.make_block_template(w, 0, 0)
        tokens = torch.from_numpy(tokens0).cuda()
        state = torch.from_numpy(state0).cuda()
        n_left = torch.from_numpy((state0 == MASKED).sum(axis=1).astype(np.int32)).cuda()
        n_comm = torch.zeros(N, dtype=torch.int32, device="cuda")
        hosts = [torch.zeros(N, dtype=torch.int32).pin_memory() for _ in range(2)]
        done = [torch.cuda.Event(), torch.cuda.Event()]
        stream = torch.cuda.current_stream()
        inputs, rec = [], []
        scale = 1.0 / np.sqrt(w.head_dim)

        def enqueue(t):
            q, k, v = synth.make_qkv(w, 0, 0, 0, t)
            lg = synth.make_logits(w, 0, 0, t, rows="all")
            inputs.append((q, k, v, lg))
            out = torch.full((q.size,), float("nan"), dtype=torch.bfloat16, device="cuda")
            fdd.fdd_block_attn_gated(ctx, [scene.forkset], 0, harness.bf16_tensor(q), harness.bf16_tensor(k),
                                     harness.bf16_tensor(v), out, [d], scale, 0, n_left)
            fdd.fdd_unmask(ctx, [scene.forkset], harness.logits_tensor(w, lg), tokens, state, [d], w.threshold,
                           w.temperature, 0, t, n_comm, n_left)
            rec.append((out, tokens.clone(), state.clone(), n_comm.clone(), n_left.clone()))
            hosts[t % 2].copy_(n_left, non_blocking=True)
            done[t % 2].record(stream)

        enqueue(0)
        t = 0
        while True:
            if t + 1 < d:
                enqueue(t + 1)
            done[t % 2].synchronize()
            left = int(hosts[t % 2].sum())
            t += 1
            if left == 0 or t >= d:
                break
        torch.cuda.synchronize()
        fdd.fdd_poll_status(ctx)
        assert 2 <= t < d and len(rec) == t + 1
        tok_in, st_in, ambiguous = tokens0, state0, 0
        for step, ((q, k, v, lg), (out, tok, st, nc, nl)) in enumerate(zip(inputs, rec)):
            decoding = np.nonzero((st_in == MASKED).any(axis=1))[0]
            got_attn = out.float().cpu().numpy().astype(np.float64).reshape(N, d, w.n_q_heads, w.head_dim)
            if len(decoding):
                ref_attn = pu.attention_oracle(w, (pk, pv), empty, q, k, v, forks=decoding)
                pu.assert_attention_close(got_attn[decoding], ref_attn)
            idle = np.setdiff1d(np.arange(N), decoding)
            assert np.all(np.isnan(got_attn[idle])), "attention wrote rows of a rollout that had finished"
            got = dict(tokens=tok.cpu().numpy(), state=st.cpu().numpy(), conf=None,
                       n_committed=nc.cpu().numpy(), n_left=nl.cpu().numpy())
            ref = unmask_step(pu.widen_logits(w, lg), tok_in, st_in, scene.seeds, w.threshold, w.temperature, 0, step)
            ambiguous += len(pu.compare_unmask(got, ref, tok_in, st_in, w.threshold)["ambiguous_forks"])
            tok_in, st_in = got["tokens"], got["state"]
        assert ambiguous <= 1
        assert not np.any(st_in == MASKED)
        assert step == t and len(decoding) == 0          # the last recorded step ran after the block was complete
    finally:
        fdd.fdd_destroy(ctx)


def test_step_recorded_as_a_cuda_graph_replays_the_block_loop():
    # One denoising step (gated attention, unmask with the step counted on the device, copy of the
    # counts) is recorded once as a CUDA graph and replayed until the block is complete; the result
    # must be what the same calls give when issued one by one with the step passed by value.
    # (This test holds the replay against the CUDA path itself; that the calls issued one by one
    # agree with the oracle is what test_pipelined_block_loop_* and test_block_loop_* check.)
    w = synth.small_variant(synth.workload("tts"), prefix_len=300, vocab=4096, n_forks=5)
    sc = w.scenes[0]
    N, d = sc.n_forks, sc.block_len
    ctx = harness.create_context(w)
    try:
        scene = harness.GpuScene(ctx, w, 0)
        tokens0, state0 = synth.make_block_template(w, 0, 0)
        q, k, v = (harness.bf16_tensor(x) for x in synth.make_qkv(w, 0, 0, 0, 0))
        lg = harness.logits_tensor(w, synth.make_logits(w, 0, 0, 0, rows="all"))   # the same inputs every step
        scale = 1.0 / np.sqrt(w.head_dim)
        n_left0 = torch.from_numpy((state0 == MASKED).sum(axis=1).astype(np.int32)).cuda()

        def eager():
            tokens, state = torch.from_numpy(tokens0).cuda(), torch.from_numpy(state0).cuda()
            n_left, n_comm = n_left0.clone(), torch.zeros(N, dtype=torch.int32, device="cuda")
            out = torch.zeros_like(q)
            trace = []
            for t in range(d):
                fdd.fdd_block_attn_gated(ctx, [scene.forkset], 0, q, k, v, out, [d], scale, 0, n_left)
                fdd.fdd_unmask(ctx, [scene.forkset], lg, tokens, state, [d], w.threshold, w.temperature, 0, t, n_comm, n_left)
                trace.append((tokens.cpu().numpy(), state.cpu().numpy(), n_left.cpu().numpy(), out.float().cpu().numpy()))
                if int(n_left.sum()) == 0:
                    break
            return trace

        ref = eager()
        assert 2 <= len(ref) < d
        # the graph: static buffers, the step index lives in `counter`
        tokens, state = torch.from_numpy(tokens0).cuda(), torch.from_numpy(state0).cuda()
        n_left, n_comm = n_left0.clone(), torch.zeros(N, dtype=torch.int32, device="cuda")
        out = torch.zeros_like(q)
        counter = torch.zeros(1, dtype=torch.int32, device="cuda")
        left_host = torch.zeros(N, dtype=torch.int32).pin_memory()
        fset, dlen = fdd.ptr_array([scene.forkset]), fdd.i32_array([d])
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                fdd.fdd_block_attn_gated(ctx, fset, 0, q, k, v, out, dlen, scale, 0, n_left)
                fdd.fdd_unmask_counted(ctx, fset, lg, tokens, state, dlen, w.threshold, w.temperature, 0, counter,
                                       n_comm, n_left)
                left_host.copy_(n_left, non_blocking=True)
        torch.cuda.current_stream().wait_stream(side)
        # capture launches nothing: reset what the block starts from and replay
        tokens.copy_(torch.from_numpy(tokens0)); state.copy_(torch.from_numpy(state0)); n_left.copy_(n_left0)
        counter.zero_()
        for t in range(len(ref)):
            graph.replay()
            torch.cuda.synchronize()
            r_tok, r_st, r_left, r_out = ref[t]
            assert np.array_equal(tokens.cpu().numpy(), r_tok) and np.array_equal(state.cpu().numpy(), r_st), t
            assert np.array_equal(left_host.numpy(), r_left) and np.array_equal(n_left.cpu().numpy(), r_left), t
            live = np.nonzero(ref[t - 1][2] if t else np.ones(N))[0]
            got_out = out.float().cpu().numpy().reshape(N, -1)
            assert np.array_equal(got_out[live], r_out.reshape(N, -1)[live]), t
            assert int(counter.item()) == t + 1
        assert int(left_host.sum()) == 0
        fdd.fdd_poll_status(ctx)
    finally:
        fdd.fdd_destroy(ctx)


def test_tts_full_size_block_loop_sampled_rollouts():
    # the test-time-scaling configuration at full size (8 rollouts, 4096-token prefix, vocabulary
    # 151936, Gumbel noise): the whole loop of one block runs on the GPU; every step the oracle
    # re-does two rollouts from the same state, and attention is checked at the first and last step
    w = synth.workload("tts")
    sc = w.scenes[0]
    ctx = harness.create_context(w)
    try:
        scene = harness.GpuScene(ctx, w, 0)
        pk, pv = synth.make_prefix(w, 0)
        empty = ([np.zeros((0, w.n_kv_heads, w.head_dim), dtype=np.uint16)] * sc.n_forks,) * 2
        tokens, state = synth.make_block_template(w, 0, 0)
        sample = [1, 6]
        step, ambiguous = 0, 0
        while np.any(state == MASKED):
            q, k, v = synth.make_qkv(w, 0, 0, 0, step)
            got_attn = pu.attention_gpu(ctx, scene, q, k, v)
            if step == 0 or int((state == MASKED).sum()) <= 3 * sc.n_forks:
                ref_attn = pu.attention_oracle(w, (pk, pv), empty, q, k, v, forks=sample)
                pu.assert_attention_close(got_attn[sample], ref_attn)
            logits = synth.make_logits(w, 0, 0, step, rows="value")
            got = pu.unmask_gpu(ctx, scene, logits, tokens, state, w.threshold, w.temperature, 0, step)
            ref = unmask_step(pu.widen_logits(w, logits[sample]), tokens[sample], state[sample], scene.seeds[sample],
                              w.threshold, w.temperature, 0, step)
            sub = {k_: v_[sample] for k_, v_ in got.items()}
            ambiguous += len(pu.compare_unmask(sub, ref, tokens[sample], state[sample], w.threshold)["ambiguous_forks"])
            assert np.all(got["n_committed"][(state == MASKED).any(axis=1)] >= 1)
            tokens, state = got["tokens"], got["state"]
            step += 1
            assert step <= sc.block_len
        assert ambiguous <= 1 and 2 <= step <= 22
        fdd.fdd_kv_commit(ctx, [scene.forkset], 0, harness.bf16_tensor(k), harness.bf16_tensor(v), [sc.block_len], 1)
        traj = synth.tokens_to_trajectory(w, tokens, state)
        out = torch.zeros((w.waypoints, 2), dtype=torch.float32, device="cuda")
        fdd.fdd_average_rollouts(ctx, torch.from_numpy(traj).cuda(), sc.n_forks, w.waypoints, out)
        fdd.fdd_poll_status(ctx)
        ref_t = average_rollouts(traj)
        assert np.all(np.abs(out.cpu().numpy() - ref_t) <= 1e-5 * np.maximum(np.abs(ref_t), 1e-30) + 1e-30)
    finally:
        fdd.fdd_destroy(ctx)


def test_average_cancellation_and_single_rollout():
    ctx = fdd.fdd_create(4, 1, 64, 64)
    try:
        g = np.random.default_rng(5)
        traj = (g.standard_normal((32, 10, 2)) * 100).astype(np.float32)
        traj[1::2] = -traj[::2] + np.float32(1e-3)        # heavy cancellation
        out = torch.zeros((10, 2), dtype=torch.float32, device="cuda")
        fdd.fdd_average_rollouts(ctx, torch.from_numpy(traj).cuda(), 32, 10, out)
        ref = average_rollouts(traj)
        got = out.cpu().numpy().astype(np.float64)
        assert np.all(np.abs(got - ref) <= 1e-5 * np.abs(ref))
        fdd.fdd_average_rollouts(ctx, torch.from_numpy(traj[:1].copy()).cuda(), 1, 10, out)
        assert np.array_equal(out.cpu().numpy(), traj[0])
    finally:
        fdd.fdd_destroy(ctx)


def test_average_after_jerk_minimising_interpolation():
    # fdd_average_rollouts_jmt against the oracle (every rollout interpolated by the library spline,
    # then averaged): the paper's 5 waypoints -> 20, the benchmark's 10 -> 40, odd sizes, one rollout,
    # rollouts that cancel, and the same call twice (the interpolation matrix is built once)
    from oracle.jmt import average_rollouts_jmt
    ctx = fdd.fdd_create(4, 1, 64, 64)
    try:
        g = np.random.default_rng(21)
        for n, w, w_out in ((4, 5, 20), (32, 10, 40), (1, 5, 20), (7, 2, 9), (3, 32, 256), (6, 10, 10), (4, 5, 20)):
            traj = np.cumsum(g.normal([4.0, 0.3], [1.5, 0.8], size=(n, w, 2)), axis=1).astype(np.float32)
            if n == 6:
                traj[3:] = -traj[:3] + np.float32(1e-3)            # cancellation: the mean is tiny
            out = torch.full((w_out, 2), float("nan"), dtype=torch.float32, device="cuda")
            fdd.fdd_average_rollouts_jmt(ctx, torch.from_numpy(traj).cuda(), n, w, w_out, out)
            fdd.fdd_poll_status(ctx)
            got = out.cpu().numpy().astype(np.float64)
            ref = average_rollouts_jmt(traj, w_out)
            scale = max(np.abs(ref).max(), 1e-30)
            assert np.all(np.abs(got - ref) <= 1e-5 * np.maximum(np.abs(ref), 1e-2 * scale)), (n, w, w_out)
        for bad in ((1, 1, 4), (1, 33, 4), (1, 5, 257)):
            with pytest.raises(fdd.FddError):
                fdd.fdd_average_rollouts_jmt(ctx, torch.zeros((bad[0], bad[1], 2), device="cuda"), bad[0], bad[1], bad[2],
                                             torch.zeros((bad[2], 2), device="cuda"))
    finally:
        fdd.fdd_destroy(ctx)


def test_upload_masked_rows_copies_exactly_the_rows_that_are_read():
    w = synth.small_variant(synth.workload("tts"), prefix_len=64, vocab=4096, n_forks=3, n_blocks=1)
    sc = w.scenes[0]
    ctx = harness.create_context(w)
    try:
        rows = sc.n_forks * sc.block_len
        g = np.random.default_rng(3)
        host = torch.from_numpy(g.integers(-30000, 30000, size=(rows, w.vocab), dtype=np.int16)).pin_memory()
        dev = torch.full((rows, w.vocab), 77, dtype=torch.int16, device="cuda")
        _, state = synth.make_block_template(w, 0, 0)
        state = state.reshape(-1).copy()
        state[5] = COMMITTED                                   # break a run of MASKED rows
        st = torch.from_numpy(state)
        n = fdd.fdd_upload_masked_rows(ctx, host, dev, st)
        torch.cuda.synchronize()
        masked = state == MASKED
        assert n == int(masked.sum()) * w.vocab * 2
        got = dev.cpu().numpy()
        assert np.array_equal(got[masked], host.numpy()[masked])
        assert np.all(got[~masked] == 77)
        assert fdd.fdd_upload_masked_rows(ctx, host, dev, torch.full((rows,), COMMITTED, dtype=torch.uint8)) == 0
    finally:
        fdd.fdd_destroy(ctx)


@pytest.mark.parametrize("vocab", [4096, 1001])
def test_pull_masked_rows_fetches_exactly_the_rows_that_are_read(vocab):
    # The same contract as the copy above, but a kernel reads the state on the device and pulls the
    # rows out of pinned host memory itself; an odd vocabulary takes the path for rows that are not
    # 16 bytes apart.
    w = synth.small_variant(synth.workload("tts"), prefix_len=64, vocab=vocab, n_forks=3, n_blocks=1)
    sc = w.scenes[0]
    ctx = harness.create_context(w)
    try:
        rows = sc.n_forks * sc.block_len
        g = np.random.default_rng(4)
        host = torch.from_numpy(g.integers(-30000, 30000, size=(rows, w.vocab), dtype=np.int16)).pin_memory()
        dev = torch.full((rows, w.vocab), 77, dtype=torch.int16, device="cuda")
        _, state = synth.make_block_template(w, 0, 0)
        state = state.reshape(-1).copy()
        state[5] = COMMITTED
        st = torch.from_numpy(state).cuda()
        count = torch.zeros(1, dtype=torch.int64, device="cuda")
        fdd.fdd_pull_masked_rows(ctx, host, dev, st, count)
        torch.cuda.synchronize()
        masked = state == MASKED
        assert int(count.item()) == int(masked.sum()) * w.vocab * 2
        got = dev.cpu().numpy()
        assert np.array_equal(got[masked], host.numpy()[masked])
        assert np.all(got[~masked] == 77)
        fdd.fdd_pull_masked_rows(ctx, host, dev, torch.full((rows,), COMMITTED, dtype=torch.uint8, device="cuda"), count)
        torch.cuda.synchronize()
        assert int(count.item()) == int(masked.sum()) * w.vocab * 2          # nothing MASKED: nothing pulled
        pageable = torch.zeros((rows, w.vocab), dtype=torch.int16)           # not pinned: the device cannot address it
        with pytest.raises(fdd.FddError) as ei:
            fdd.fdd_pull_masked_rows(ctx, pageable, dev, st, None)
        assert ei.value.status == fdd.FDD_ERR_INVALID_ARG
        fdd.fdd_poll_status(ctx)
    finally:
        fdd.fdd_destroy(ctx)


# ---------------------------------------------------------------------------------------------
# host-side error paths (nothing is launched)
# ---------------------------------------------------------------------------------------------
def test_error_paths():
    with pytest.raises(fdd.FddError) as ei:
        fdd.fdd_create(16, 2, 96, 1000)
    assert ei.value.status == fdd.FDD_ERR_UNSUPPORTED
    with pytest.raises(fdd.FddError):
        fdd.fdd_create(16, 3, 128, 1000)
    w = synth.small_variant(synth.workload("tts"), prefix_len=64, vocab=512, n_forks=2, n_blocks=1)
    ctx = harness.create_context(w)
    try:
        scene = harness.GpuScene(ctx, w, 0)
        q, k, v = (harness.bf16_tensor(x) for x in synth.make_qkv(w, 0, 0, 0, 0))
        out = torch.empty_like(q)
        with pytest.raises(fdd.FddError) as ei:
            fdd.fdd_block_attn(ctx, [scene.forkset], 0, q, k, v, out, [w.scenes[0].block_len + 100], 0.1)
        assert ei.value.status == fdd.FDD_ERR_CAPACITY
        with pytest.raises(fdd.FddError) as ei:
            fdd.fdd_block_attn(ctx, [scene.forkset], 3, q, k, v, out, [32], 0.1)
        assert ei.value.status == fdd.FDD_ERR_SHAPE
        with pytest.raises(fdd.FddError) as ei:
            fdd.fdd_block_attn(ctx, [scene.forkset], 0, None, k, v, out, [32], 0.1)
        assert ei.value.status == fdd.FDD_ERR_INVALID_ARG
        with pytest.raises(fdd.FddError) as ei:
            fdd.fdd_fork(ctx, scene.prefix_k, scene.prefix_v, None, 64, 64, 999, [1] * 999,
                         scene.suffix_k, scene.suffix_v, 32)
        assert ei.value.status == fdd.FDD_ERR_CAPACITY
        fs = scene.forkset
        scene.free()
        with pytest.raises(fdd.FddError) as ei:           # freed handle
            fdd.fdd_block_attn(ctx, [fs], 0, q, k, v, out, [32], 0.1)
        assert ei.value.status == fdd.FDD_ERR_STATE
        with pytest.raises(fdd.FddError) as ei:           # double free
            fdd.fdd_forkset_free(ctx, fs)
        assert ei.value.status == fdd.FDD_ERR_STATE
        assert "not live" in fdd.fdd_last_error(ctx)
        assert fdd.fdd_poll_status(ctx) == fdd.FDD_OK
    finally:
        fdd.fdd_destroy(ctx)
