"""Benchmark of the block-diffusion decode hot path on B200.

One "step" decodes one section block for every rollout of the scene:
    fdd_fork -> repeat { fdd_block_attn x layers ; fdd_unmask ; read n_left } until no
    MASKED position is left -> fdd_kv_commit x layers -> fdd_average_rollouts.
Metric: committed (value) tokens per second over all rollouts.  Inputs are seeded synthetic
tensors shaped like the paper's driving workload (see paper_2605_23163_b200/synth.py).

    python bench.py --gpus 1 --steps 10 --warmup 3            # this implementation
    python bench.py --impl reference --steps 2 --warmup 1      # the CPU fp64 oracle, timed
Under torchrun (N > 1) every rank decodes an independent scene replica (no data-path
collective); the time is the max over ranks and the value the sum of all ranks' tokens.
"""
import argparse
import ctypes
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "committed tokens/s per denoise step (N forks, shared prefix)"
UNIT = "tokens/s"
TIMED_PASSES = 3    # the timed region (exactly --steps blocks) is run this often; the median pass is reported
COUNT_STREAM = None  # copy the per-rollout counts to the host on a stream of their own (None: for large steps only)
GRAPH = False       # replay every denoising step from a CUDA graph (--graph)
TIME_EVERY = 20     # blocks between two blocks whose kernels are timed one by one
NATIVE_LOOP = True  # the block loop is run by the library (fdd_decode_block); --loop python keeps it in this file
LOOKAHEAD = True   # enqueue step t + 1 before the host has read the counts of step t (--no-lookahead)
PRE_STEPS = 6      # distinct per-step input sets kept resident; later steps cycle through them (--pre-steps)


def _kernel_source_hash(names):
    """sha256 over the named kernel sources: ties a stored counter to the code it was taken from."""
    import hashlib
    h = hashlib.sha256()
    for n in names:
        with open(os.path.join(ROOT, "paper_2605_23163_b200", "csrc", n), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def _stored_traffic(workload):
    """DRAM bytes (read + write) per attention launch from the tracked ncu summary of this workload, or
    None when there is none or the kernel's source has changed since the counters were taken."""
    path = os.path.join(ROOT, "profiles", f"attn_ptc_{workload}.md")
    if not os.path.exists(path):
        return None
    import re
    text = open(path).read()
    m_b = re.search(r"dram_bytes_per_launch:\s*([0-9.eE+]+)", text)
    m_h = re.search(r"kernel_source_sha256:\s*([0-9a-f]{64})", text)
    m_d = re.search(r"captured:\s*(\S+)", text)
    if not (m_b and m_h) or m_h.group(1) != _kernel_source_hash(["attn_ptc.cu", "tc_ptx.cuh"]):
        return None
    return {"bytes": float(m_b.group(1)), "captured": m_d.group(1) if m_d else None}


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.stop_flag = index, [], set(), False
        self.max_mhz = None

    def run(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            h = nv.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM)
            names = {
                getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
                getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
                getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
                getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
            }
            while not self.stop_flag:
                self.samples.append(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
                time.sleep(0.004)
        except Exception as exc:      # NVML unavailable: report that instead of clocks
            self.reasons.add(f"nvml_unavailable:{type(exc).__name__}")

    def summary(self):
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def _gen_step_inputs(w, scene_idx, block, step, pool):
    """numpy inputs of one denoising step: q/k/v bits and logits (value rows only)."""
    from paper_2605_23163_b200 import synth
    q, k, v = synth.make_qkv(w, scene_idx, 0, block, step)
    sc = w.scenes[scene_idx]
    dt = np.uint16 if w.logits_dtype == "bf16" else np.float32
    logits = np.zeros((sc.n_forks, sc.block_len, w.vocab), dtype=dt)
    frozen = set(synth.scaffold_positions(w, scene_idx, block).tolist())
    jobs = [(f, i) for f in range(sc.n_forks) for i in range(sc.block_len) if i not in frozen]

    def fill(job):
        f, i = job
        logits[f, i] = synth.make_logits_row(w, scene_idx, block, step, f, i)

    list(pool.map(fill, jobs))
    return q, k, v, logits


def _attn_flops(w, sc, suffix_len):
    return 4.0 * sc.n_forks * sc.block_len * w.n_q_heads * (sc.prefix_len + suffix_len + sc.block_len) * w.head_dim


def run_ours(args):
    import torch
    from concurrent.futures import ThreadPoolExecutor
    from paper_2605_23163_b200 import fdd, harness, replicas, synth

    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    fdd.lib()
    w = synth.workload(args.workload)
    if args.n_forks:                           # rollout sweep: same shapes, another number of rollouts
        w = synth.small_variant(w, n_forks=args.n_forks, name=w.name)
    w = replicas.replica_workload(w, rank)     # every rank decodes its own scene (different seed)
    # A workload is one scene or a batch of independent scenes (the serving mix): every call below
    # takes all of them at once, packed in scene order.
    n_scenes = len(w.scenes)
    sc = w.scenes[0]
    L = args.layers
    ctx = harness.create_context(w, n_layers=L)
    gscenes = [harness.GpuScene(ctx, w, i, n_layers=L, suffix_capacity=w.scenes[i].block_len) for i in range(n_scenes)]
    for g in gscenes:                      # the benchmark forks anew for every block
        g.free()
    stream = torch.cuda.current_stream()
    stream_c = ctypes.c_void_p(stream.cuda_stream)
    scale = 1.0 / np.sqrt(w.head_dim)
    ds = [s_.block_len for s_ in w.scenes]
    Ns = [s_.n_forks for s_ in w.scenes]
    d, N = max(ds), sum(Ns)

    pool = ThreadPoolExecutor(max_workers=max(1, len(os.sched_getaffinity(0))))
    host_steps = []
    for t in range(PRE_STEPS):
        per_scene = [_gen_step_inputs(w, i, 0, t, pool) for i in range(n_scenes)]
        host_steps.append(tuple(np.concatenate([x[j].reshape(-1) for x in per_scene]) for j in range(4)))
    pool.shutdown()
    dev_steps = []
    for q, k, v, lg in host_steps:
        dev_steps.append(tuple([harness.bf16_tensor(q), harness.bf16_tensor(k), harness.bf16_tensor(v),
                                harness.logits_tensor(w, lg)]))
    templates = [synth.make_block_template(w, i, 0) for i in range(n_scenes)]
    tokens0 = np.concatenate([t_.reshape(-1) for t_, _ in templates])
    state0 = np.concatenate([s_.reshape(-1) for _, s_ in templates])
    tokens0_d = torch.from_numpy(tokens0).cuda()
    state0_d = torch.from_numpy(state0).cuda()
    # tokens and state of the block live in one buffer (and their templates in another of the same
    # layout), so that a block starts with one copy
    blk0 = torch.cat([tokens0_d.view(torch.uint8), state0_d])
    blk = torch.empty_like(blk0)
    tokens = blk[:tokens0_d.numel() * 4].view(torch.int32)
    state = blk[tokens0_d.numel() * 4:]
    out = torch.empty_like(dev_steps[0][0])
    n_comm = torch.zeros(N, dtype=torch.int32, device="cuda")
    n_left = torch.zeros(N, dtype=torch.int32, device="cuda")
    n_left_host = torch.zeros(N, dtype=torch.int32).pin_memory()
    trajs = [torch.from_numpy(synth.tokens_to_trajectory(w, t_, s_)).cuda() for t_, s_ in templates]
    traj_out = torch.zeros((n_scenes, w.waypoints, 2), dtype=torch.float32, device="cuda")
    value_tokens = int((state0 == synth.MASKED).sum())
    all_tokens = int(state0.size)

    # MASKED positions per rollout at the start of a block: the gate of the first attention call
    n_left0_d = torch.from_numpy(np.concatenate(
        [(s_ == synth.MASKED).sum(axis=1).astype(np.int32) for _, s_ in templates])).cuda()
    n_left_hosts = [torch.zeros(N, dtype=torch.int32).pin_memory() for _ in range(2)]
    n_left_views = [t_.numpy() for t_ in n_left_hosts]          # the host reads the counts through these
    # arguments that are the same in every call are marshalled once
    ds_c = fdd.i32_array(ds)
    fork_args = [(fdd.ptr_array(g.prefix_k), fdd.ptr_array(g.prefix_v), g.page_table, g.sc.prefix_len,
                  g.prefix_capacity, g.sc.n_forks, fdd.u64_array(g.seeds), fdd.ptr_array(g.suffix_k),
                  fdd.ptr_array(g.suffix_v), g.suffix_capacity) for g in gscenes]
    step_done = [torch.cuda.Event(), torch.cuda.Event()]
    # The counts go to the host on a stream of their own, so that the next attention call does not
    # queue behind the copy; unmask writes them to two device buffers in turn (step t + 2 reuses the
    # buffer of step t, whose copy the host has waited for by then).
    count_stream = torch.cuda.Stream()
    # (worth it when a step's kernels are long; a latency-bound step loses more to the second stream's
    # event than the copy costs in line)
    use_count_stream = COUNT_STREAM if COUNT_STREAM is not None else all_tokens >= 1024
    unmask_done = [torch.cuda.Event(), torch.cuda.Event()]
    n_left_d = [n_left, torch.zeros_like(n_left)]

    prepared, retired = [], []  # fork sets made ahead for the next block / of the last block, to be freed
    attn_events = []            # [start, end, rollouts still decoding] of every timed attention call
    unmask_events = []          # [start, end, MASKED rows on entry] of every timed unmask call

    def decode_block(inputs, timed_attn, lookahead):
        """One step of the benchmark: the whole block loop for all rollouts.  `inputs(t)` returns
        device tensors (q, k, v, logits) of denoising step t.  Attention is gated by the n_left
        array of the step before, so rollouts that have finished their block cost nothing; with
        `lookahead` step t + 1 is enqueued before the host has seen the result of step t (once
        every rollout is done its kernels return at once), which keeps the GPU busy while the host
        reads the counts."""
        # The fork sets of this block were made while the block before was running (fdd_fork is host
        # work only), and the sets of the block before are freed once this block's first step is
        # enqueued: neither sits between two blocks, where the GPU would wait for the host.
        fs_list = prepared.pop() if prepared else [fdd.fdd_fork(ctx, *fa) for fa in fork_args]
        fs = fdd.ptr_array(fs_list)
        tokens.copy_(tokens0_d, non_blocking=True)
        state.copy_(state0_d, non_blocking=True)
        kv_of = [None, None]
        pending = [None, None]      # the event records of a step, completed once its entry counts are known

        def enqueue(t):
            q, k, v, lg, *after = inputs(t)       # (after: an event the logits are ready behind, if they come by another stream)
            kv_of[t % 2] = (k, v)
            gate = n_left0_d if t == 0 else n_left_d[(t - 1) % 2]     # who still decodes: the counts of the step before
            recs = []
            for layer in range(L):
                if timed_attn:
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record(stream)
                fdd.fdd_block_attn_gated(ctx, fs, layer, q, k, v, out, ds_c, scale, 0, gate)
                if timed_attn:
                    e1.record(stream)
                    recs.append([e0, e1, None])
                    attn_events.append(recs[-1])
            if timed_attn:
                u0, u1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                u0.record(stream)
            if after:
                stream.wait_event(after[0])
            fdd.fdd_unmask(ctx, fs, lg, tokens, state, ds_c, w.threshold, w.temperature, 0, t, n_comm, n_left_d[t % 2])
            if timed_attn:
                u1.record(stream)
                recs.append([u0, u1, None])
                unmask_events.append(recs[-1])
            if use_count_stream:
                unmask_done[t % 2].record(stream)
                count_stream.wait_event(unmask_done[t % 2])
                with torch.cuda.stream(count_stream):
                    n_left_hosts[t % 2].copy_(n_left_d[t % 2], non_blocking=True)
                    step_done[t % 2].record(count_stream)
            else:
                n_left_hosts[t % 2].copy_(n_left_d[t % 2], non_blocking=True)
                step_done[t % 2].record(stream)
            pending[t % 2] = recs

        def entry_counts(t, rollouts, rows):
            for r in pending[t % 2][:-1]:
                r[2] = rollouts
            if pending[t % 2]:
                pending[t % 2][-1][2] = rows

        enqueue(0)
        entry_counts(0, N, value_tokens)
        while retired:
            for f_ in retired.pop():
                fdd.fdd_forkset_free(ctx, f_)
        t = 0
        while True:
            if lookahead and t + 1 < d:
                enqueue(t + 1)
            if t == 0:
                prepared.append([fdd.fdd_fork(ctx, *fa) for fa in fork_args])     # for the next block
            step_done[t % 2].synchronize()
            left = n_left_views[t % 2]
            masked_rows = int(left.sum())
            t += 1
            if lookahead and t < d:
                entry_counts(t, int((left != 0).sum()), masked_rows)
            if masked_rows == 0 or t >= d:
                break
            if not lookahead:
                enqueue(t)
                entry_counts(t, int((left != 0).sum()), masked_rows)
        k, v = kv_of[(t - 1) % 2]
        for layer in range(L):
            fdd.fdd_kv_commit(ctx, fs, layer, k, v, ds_c, 1 if layer == L - 1 else 0)
        for i in range(n_scenes):
            fdd.fdd_average_rollouts(ctx, trajs[i], Ns[i], w.waypoints, traj_out[i])
        retired.append(fs_list)
        return t

    resident = lambda t: dev_steps[t % PRE_STEPS]

    # ---- the same loop with every denoising step replayed from a CUDA graph (--graph).  A graph holds
    # the L gated attention calls, the unmask call with the step counted on the device and the copy
    # of the counts; there is one graph per resident input set (their addresses are part of it).
    # The fork sets are made once and start every block with fdd_forkset_reset.
    g_graphs = {}
    g_period = PRE_STEPS if PRE_STEPS % 2 == 0 else 2 * PRE_STEPS      # input set and host count buffer of step t
    g_n_left = torch.zeros_like(n_left)
    g_counter = torch.zeros(1, dtype=torch.int32, device="cuda")
    g_sets = {"list": None, "arr": None}
    g_replays = [0]
    capture_stream = torch.cuda.Stream()

    def graph_of(t):
        key = t % g_period
        if key not in g_graphs:
            q, k, v, lg = resident(t)
            gph = torch.cuda.CUDAGraph()
            capture_stream.wait_stream(stream)
            with torch.cuda.stream(capture_stream):
                with torch.cuda.graph(gph, stream=capture_stream):
                    for layer in range(L):
                        fdd.fdd_block_attn_gated(ctx, g_sets["arr"], layer, q, k, v, out, ds_c, scale, 0, g_n_left)
                    fdd.fdd_unmask_counted(ctx, g_sets["arr"], lg, tokens, state, ds_c, w.threshold, w.temperature, 0,
                                           g_counter, n_comm, g_n_left)
                    n_left_hosts[t % 2].copy_(g_n_left, non_blocking=True)
            stream.wait_stream(capture_stream)
            g_graphs[key] = gph
        return g_graphs[key]

    def decode_block_graph():
        if g_sets["list"] is None:
            g_sets["list"] = [fdd.fdd_fork(ctx, *fa) for fa in fork_args]
            g_sets["arr"] = fdd.ptr_array(g_sets["list"])
        else:
            for f_ in g_sets["list"]:
                fdd.fdd_forkset_reset(ctx, f_)
        tokens.copy_(tokens0_d, non_blocking=True)
        state.copy_(state0_d, non_blocking=True)
        g_n_left.copy_(n_left0_d, non_blocking=True)
        g_counter.zero_()

        def replay(t):
            graph_of(t).replay()
            step_done[t % 2].record(stream)
            g_replays[0] += 1

        replay(0)
        t = 0
        while True:
            if t + 1 < d:
                replay(t + 1)
            step_done[t % 2].synchronize()
            masked_rows = int(n_left_views[t % 2].sum())
            t += 1
            if masked_rows == 0 or t >= d:
                break
        _, k, v, _ = resident(t - 1)
        for layer in range(L):
            fdd.fdd_kv_commit(ctx, g_sets["arr"], layer, k, v, ds_c, 1 if layer == L - 1 else 0)
        for i in range(n_scenes):
            fdd.fdd_average_rollouts(ctx, trajs[i], Ns[i], w.waypoints, traj_out[i])
        return t

    # ---- the same loop run by the library (fdd_decode_block): the calls of a step are issued from
    # native code, one step ahead of the counts, and the block's K/V are committed by the same call.
    # The fork sets are made once and start every block with fdd_forkset_reset.
    nat = {"list": None, "arr": None, "call": None, "avg": None}
    nat_q = fdd.ptr_array([dev_steps[t][0] for t in range(PRE_STEPS) for _ in range(L)])
    nat_k = fdd.ptr_array([dev_steps[t][1] for t in range(PRE_STEPS) for _ in range(L)])
    nat_v = fdd.ptr_array([dev_steps[t][2] for t in range(PRE_STEPS) for _ in range(L)])
    nat_out = fdd.ptr_array([out for t in range(PRE_STEPS) for _ in range(L)])
    nat_lg = fdd.ptr_array([dev_steps[t][3] for t in range(PRE_STEPS)])

    def decode_block_native():
        if nat["list"] is None:
            nat["list"] = [fdd.fdd_fork(ctx, *fa) for fa in fork_args]
            nat["arr"] = fdd.ptr_array(nat["list"])
            # (the same call block after block: its arguments are marshalled once)
            nat["call"] = fdd.decode_block_call(ctx, nat["arr"], L, d, nat_q, nat_k, nat_v, nat_out, nat_lg, tokens, state,
                                                ds_c, scale, 0, w.threshold, w.temperature, 0, 1, n_comm, n_left,
                                                stream=stream_c)
            nat["avg"] = [fdd.average_rollouts_call(ctx, trajs[i], Ns[i], w.waypoints, traj_out[i], stream=stream_c)
                          for i in range(n_scenes)]
        else:
            for f_ in nat["list"]:
                fdd.fdd_forkset_reset(ctx, f_)
        blk.copy_(blk0, non_blocking=True)
        steps, left = nat["call"]()
        assert left == 0
        for avg in nat["avg"]:
            avg()
        return steps

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        n_denoise = decode_block(resident, False, LOOKAHEAD)
    if GRAPH:
        for _ in range(2):                   # records the graphs of the steps a block usually takes
            decode_block_graph()
    if NATIVE_LOOP:
        for _ in range(2):
            decode_block_native()
    sampler = ClockSampler(local)
    sampler.start()
    # every TIME_EVERY-th block carries CUDA events around each of its kernels (the per-kernel
    # durations of the roofline figures); the others run as a user would run them.  The timed
    # region (exactly --steps blocks between two events) is run TIMED_PASSES times; the pass with
    # the median duration is the one reported.
    passes = []
    for _pass in range(TIMED_PASSES):
        barrier()
        launches0 = fdd.fdd_launch_count(ctx)
        replays0 = g_replays[0]
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(stream)
        denoise_steps = 0
        timed_blocks = 0
        for b_ in range(args.steps):
            per_kernel = TIME_EVERY > 0 and b_ % TIME_EVERY == 0
            timed_blocks += per_kernel
            if GRAPH and not per_kernel:
                denoise_steps += decode_block_graph()
            elif NATIVE_LOOP and not per_kernel:
                denoise_steps += decode_block_native()
            else:
                denoise_steps += decode_block(resident, per_kernel, LOOKAHEAD)
        ev1.record(stream)
        barrier()
        launches = fdd.fdd_launch_count(ctx) - launches0
        launches += (g_replays[0] - replays0) * (L + 2)  # a replayed step launches L attention kernels and the unmask pair
        passes.append(dict(ms=ev0.elapsed_time(ev1), launches=launches, denoise_steps=denoise_steps, timed_blocks=timed_blocks))
    sampler.stop_flag = True
    sampler.join(timeout=2)
    timed_blocks *= TIMED_PASSES                     # the per-kernel events of all passes are pooled
    chosen = sorted(passes, key=lambda p_: p_["ms"])[len(passes) // 2]
    ms, launches, denoise_steps = chosen["ms"], chosen["launches"], chosen["denoise_steps"]
    attn_all = [(a.elapsed_time(b), n) for a, b, n in attn_events]
    rollout_steps = sum(n for _, n in attn_all) / L     # (rollout, step) pairs that decoded
    attn_ms = [ms_ for ms_, n in attn_all if n == N]          # launches in which every rollout decodes
    unmask_ms = [(a.elapsed_time(b), rows) for a, b, rows in unmask_events]
    ms = replicas.max_over_ranks(ms, dist, "cuda")
    fdd.fdd_poll_status(ctx)

    # The same first-step unmask launch without noise (temperature 0, the deterministic sections):
    # every value row MASKED, one launch per resident input set in turn (together larger than L2).
    fs_list = [fdd.fdd_fork(ctx, *fa) for fa in fork_args]
    fs_arr = fdd.ptr_array(fs_list)
    greedy_ev = []
    for it in range(3 + 2 * PRE_STEPS):              # enqueued back to back: the GPU never waits for the host in between
        lg = dev_steps[it % PRE_STEPS][3]
        tokens.copy_(tokens0_d, non_blocking=True)
        state.copy_(state0_d, non_blocking=True)
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record(stream)
        fdd.fdd_unmask(ctx, fs_arr, lg, tokens, state, ds_c, w.threshold, 0.0, 0, 0, n_comm, n_left)
        g1.record(stream)
        greedy_ev.append((g0, g1))
    stream.synchronize()
    greedy_ms = [a.elapsed_time(b) for a, b in greedy_ev[3:]]

    # Parity on a sample, with the counts the acceptance rule asks for: the first unmasking step of the
    # first rollouts of scene 0, GPU against the CPU oracle on the same inputs (rank 0, one GPU only).
    parity = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        parity = parity_sample(w, ctx, fs_list[0], host_steps[0][3], dev_steps[0][3], templates[0], gscenes[0].seeds,
                               tokens, state, tokens0_d, state0_d, fs_arr, ds_c, n_comm, n_left, budget_s=args.cpu_budget / 2)
    for f_ in fs_list:
        fdd.fdd_forkset_free(ctx, f_)

    # end to end: every denoising step's inputs come from pinned host memory, results go back
    e2e = None
    if not args.no_e2e:
        pinned = [tuple(torch.from_numpy(np.ascontiguousarray(a).view(np.int16) if a.dtype == np.uint16 else a).pin_memory()
                        for a in hs) for hs in host_steps]
        stage = [torch.empty_like(x) for x in dev_steps[0]]
        tok_host = torch.zeros_like(tokens0_d, device="cpu").pin_memory()
        traj_host = torch.zeros((n_scenes, w.waypoints, 2), dtype=torch.float32).pin_memory()
        d2h_step = n_left_host.numel() * 4

        pulled = torch.zeros(1, dtype=torch.int64, device="cuda")
        qkv_bytes = [0]

        def from_host(t):
            """q, k, v in full (copies); of the logits only the rows the method reads (MASKED positions),
            which a kernel pulls out of the pinned host buffer after reading the state on the device:
            nothing is read back and nothing waits on the host."""
            src = pinned[t % PRE_STEPS]
            for dst, s_ in zip(stage[:3], src[:3]):
                dst.view(torch.int16).copy_(s_, non_blocking=True)
                qkv_bytes[0] += s_.numel() * s_.element_size()
            fdd.fdd_pull_masked_rows(ctx, src[3], stage[3], state, pulled)
            return tuple(stage)

        e2e_steps = max(1, min(args.steps, args.e2e_steps))
        decode_block(from_host, False, False)
        barrier()
        ee0, ee1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ee0.record(stream)
        e2e_denoise = 0
        qkv_bytes[0] = 0
        pulled.zero_()
        for _ in range(e2e_steps):
            e2e_denoise += decode_block(from_host, False, False)     # (no step ahead: its q, k, v would cross the link for nothing)
            tok_host.copy_(tokens, non_blocking=True)
            traj_host.copy_(traj_out, non_blocking=True)
            stream.synchronize()
        ee1.record(stream)
        barrier()
        e_ms = ee0.elapsed_time(ee1)
        e_ms = replicas.max_over_ranks(e_ms, dist, "cuda")
        per_block_denoise = e2e_denoise / e2e_steps
        e2e = {"value": world * value_tokens * e2e_steps / (e_ms * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": int((qkv_bytes[0] + int(pulled.item())) / e2e_steps),
               "d2h_bytes_per_step": int(d2h_step * per_block_denoise + tok_host.numel() * 4 + traj_host.numel() * 4),
               "steps": e2e_steps, "ms_per_step": e_ms / e2e_steps}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    peaks = _peaks()
    clocks = sampler.summary()
    # Which measured bf16 peak the attention kernel is held against: the burst figure (a matmul timed
    # alone) unless the clock samples of this run show the capped state the sustained figure was taken in.
    capped = "sw_power_cap" in clocks["reasons"] and clocks["sm_mhz"] is not None and clocks["sm_max_mhz"] \
        and clocks["sm_mhz"] < 0.9 * clocks["sm_max_mhz"]
    tensor_peak = peaks["bf16_tflops_sustained"] if capped else peaks["bf16_tflops"]
    flops = sum(_attn_flops(w, s_, 0) for s_ in w.scenes)
    attn_avg_ms = float(np.mean(attn_ms)) if attn_ms else None
    achieved = flops / (attn_avg_ms * 1e-3) / 1e12 if attn_avg_ms else None
    # unmask: the launches that see every value row MASKED (first denoising step of a block)
    esz = 2 if w.logits_dtype == "bf16" else 4
    first = [ms_ for ms_, rows in unmask_ms if rows == value_tokens]
    um_ms = float(np.mean(first)) if first else None
    um_bytes = float(value_tokens) * w.vocab * esz
    um_gbs = um_bytes / (um_ms * 1e-3) / 1e9 if um_ms else None
    greedy_avg_ms = float(np.mean(greedy_ms)) if greedy_ms else None
    greedy_gbs = um_bytes / (greedy_avg_ms * 1e-3) / 1e9 if greedy_avg_ms else None
    traffic = _stored_traffic(args.workload) if L == 1 and not args.n_forks else None
    line = {
        "metric": METRIC, "value": world * value_tokens * args.steps / (ms * 1e-3), "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": args.workload, "scenes": n_scenes, "n_forks": N, "block_len": d,
                   "prefix_len": sc.prefix_len if n_scenes == 1 else [s_.prefix_len for s_ in w.scenes],
                   "heads": f"{w.n_q_heads}q/{w.n_kv_heads}kv", "head_dim": w.head_dim, "vocab": w.vocab,
                   "layers": L, "threshold": w.threshold, "temperature": w.temperature,
                   "denoise_steps_per_block": denoise_steps / args.steps,
                   # value tokens a rollout commits per denoising step it takes part in (the paper's Tok/Step)
                   "tokens_per_step_per_rollout": (value_tokens * timed_blocks / rollout_steps) if rollout_steps else None,
                   "value_tokens_per_block": value_tokens, "tokens_incl_scaffold_per_block": all_tokens,
                   "l2": "per-step inputs (logits) larger than L2",
                   "step_pipeline": ("attention gated by n_left; step t+1 enqueued before the host reads step t"
                                     if LOOKAHEAD else "attention gated by n_left; one step in flight"),
                   "steps_from_cuda_graph": bool(GRAPH),
                   "block_loop": ("library (fdd_decode_block)" if NATIVE_LOOP and not GRAPH else "bench.py"),
                   "blocks_timed_kernel_by_kernel": (f"one in {TIME_EVERY}" if TIME_EVERY else "none"),
                   "count_copy": "own stream" if use_count_stream else "compute stream",
                   "rollouts_decoding_per_attention_call": float(np.mean([n for _, n in attn_all])) if attn_all else None,
                   "replicas": "independent scene per GPU, no collective"},
        "clocks": clocks,
        "e2e": e2e,
        "gpu_launches": int(launches),
        "roofline": {"kernel": "fdd_block_attn (attn_ptc_kernel)", "bound": "tensor", "achieved": achieved,
                     "peak": tensor_peak, "unit": "TFLOP/s",
                     "frac": (achieved / tensor_peak) if achieved else None,
                     "traffic": traffic["bytes"] if traffic else None,
                     "traffic_source": (f"ncu capture of {traffic['captured']}, profiles/attn_ptc_{args.workload}.md"
                                        if traffic else "none for this kernel source and workload"),
                     "peak_source": peaks["source"] + (" (sustained bf16: the clock samples show the power-capped state)"
                                                       if capped else " (burst bf16: clocks at maximum, no power cap sampled)"),
                     "frac_of_burst_peak": (achieved / peaks["bf16_tflops"]) if achieved else None,
                     "frac_of_sustained_peak": (achieved / peaks["bf16_tflops_sustained"]) if achieved else None,
                     "launch_ms_x_sm_mhz": (attn_avg_ms * clocks["sm_mhz"]) if attn_avg_ms and clocks["sm_mhz"] else None,
                     "flops_per_launch": flops, "avg_launch_ms": attn_avg_ms, "launches_timed": len(attn_ms),
                     "blocks_timed_per_kernel": int(timed_blocks),
                     "launches": "those in which every rollout still decodes (first step of a block)",
                     "avg_ms_all_launches": float(np.mean([ms_ for ms_, _ in attn_all])) if attn_all else None},
        "roofline_unmask": {"kernel": "fdd_unmask (unmask_stream_kernel + unmask_finalize_kernel), first step of a block: "
                                      "every value row MASKED, temperature %g" % w.temperature,
                            "bound": "hbm", "achieved": um_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                            "frac": (um_gbs / peaks["hbm_gbs"]) if um_gbs else None,
                            "bytes_per_launch": um_bytes, "avg_launch_ms": um_ms, "launches_timed": len(first),
                            "peak_source": peaks["source"]},
        "roofline_unmask_greedy": {"kernel": "fdd_unmask, the same rows at temperature 0 (no noise)", "bound": "hbm",
                                   "achieved": greedy_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                   "frac": (greedy_gbs / peaks["hbm_gbs"]) if greedy_gbs else None,
                                   "bytes_per_launch": um_bytes, "avg_launch_ms": greedy_avg_ms,
                                   "launches_timed": len(greedy_ms), "peak_source": peaks["source"]},
        "parity_sample": parity,
        "timed_passes": [p_["ms"] for p_ in passes],
        "tokens_per_s_incl_scaffold": world * all_tokens * args.steps / (ms * 1e-3),
    }
    if not args.no_cpu_baseline and world >= 1:
        line["cpu_baseline"] = cpu_baseline(args.workload, budget_s=args.cpu_budget)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


# -------------------------------------------------------------------------------------------------
# CPU oracle legs
# -------------------------------------------------------------------------------------------------
def _oracle_block(w, fork, max_steps=None):
    """Decode one block for a single rollout with the CPU oracle; returns (seconds, committed
    value tokens, denoising steps)."""
    from oracle.cache import ForkSet
    from oracle.decode import decode_block
    from oracle.attention import bf16_bits_to_f64
    from paper_2605_23163_b200 import synth
    sc = w.scenes[0]
    pk, pv = synth.make_prefix(w, 0)
    seeds = synth.fork_seeds(w, 0)[fork:fork + 1]
    fs = ForkSet([pk], [pv], 1, seeds)
    tokens, state = synth.make_block_template(w, 0, 0)
    tokens, state = tokens[fork:fork + 1], state[fork:fork + 1]
    frozen = set(synth.scaffold_positions(w, 0, 0).tolist())
    cache = {}

    def inputs(t):
        if t not in cache:
            q, k, v = synth.make_qkv(w, 0, 0, 0, t)
            lg = np.zeros((1, sc.block_len, w.vocab), dtype=np.float64)
            for i in range(sc.block_len):
                if i not in frozen:
                    row = synth.make_logits_row(w, 0, 0, t, fork, i)
                    lg[0, i] = bf16_bits_to_f64(row) if w.logits_dtype == "bf16" else row
            cache[t] = dict(q=[q[fork:fork + 1]], k=[k[fork:fork + 1]], v=[v[fork:fork + 1]], logits=lg)
        return cache[t]

    for t in range(PRE_STEPS):       # inputs are made outside the timed region
        inputs(t)
    t0 = time.perf_counter()
    r = decode_block(fs, lambda t: inputs(t % PRE_STEPS), tokens, state, w.threshold, w.temperature, 0,
                     1.0 / np.sqrt(w.head_dim), max_steps=max_steps)
    dt = time.perf_counter() - t0
    return dt, int(sum(int(c.sum()) for c in r["committed_per_step"])), r["steps"]


def parity_sample(w, ctx, forkset, host_logits, dev_logits, template, seeds, tokens, state, tokens0_d, state0_d,
                  fs_arr, ds_c, n_comm, n_left, budget_s=10.0):
    """First unmasking step of the first rollouts of scene 0 on the GPU and in the CPU oracle: how many
    rows were compared, how many have a top-two score margin of at most 1e-3 (counted, not compared),
    how many rollouts are ambiguous (a confidence within 1e-4 of the threshold, or a low-margin commit),
    and how many clear rows or rollouts disagree (must be 0)."""
    import torch
    from oracle.unmask import unmask_step
    from oracle.attention import bf16_bits_to_f64
    from paper_2605_23163_b200 import fdd, synth
    sc = w.scenes[0]
    tok0, st0 = template
    N, d = tok0.shape
    tokens.copy_(tokens0_d)
    state.copy_(state0_d)
    fdd.fdd_unmask(ctx, fs_arr, dev_logits, tokens, state, ds_c, w.threshold, w.temperature, 0, 0, n_comm, n_left)
    torch.cuda.synchronize()
    got_tok = tokens.cpu().numpy()[:N * d].reshape(N, d)
    got_st = state.cpu().numpy()[:N * d].reshape(N, d)
    lg = np.asarray(host_logits).reshape(-1, w.vocab)[:N * d].reshape(N, d, w.vocab)
    rows = low = ambiguous = mismatched_rows = mismatched_rollouts = checked = 0
    t0 = time.perf_counter()
    for f in range(N):
        if f > 0 and time.perf_counter() - t0 > budget_s:
            break
        l64 = bf16_bits_to_f64(lg[f:f + 1]) if w.logits_dtype == "bf16" else lg[f:f + 1].astype(np.float64)
        ref = unmask_step(l64, tok0[f:f + 1], st0[f:f + 1], seeds[f:f + 1], w.threshold, w.temperature, 0, 0)
        masked = st0[f] == synth.MASKED
        margin = ref["score_margin"][0]
        conf = ref["conf"][0]
        rows += int(masked.sum())
        low += int((masked & (margin <= 1e-3)).sum())
        committed_ref = masked & (ref["state"][0] != synth.MASKED)
        amb = bool(np.any(np.abs(conf[masked] - w.threshold) < 1e-4)) or bool(np.any(margin[committed_ref] <= 1e-3))
        if ref["fallback"][0] and masked.sum() > 1:           # the at-least-one pick between two near-equal confidences
            top2 = np.sort(conf[masked])[-2:]
            amb = amb or bool(top2[1] - top2[0] < 1e-4 * max(top2[1], 1e-30))
        ambiguous += int(amb)
        both = masked & (got_st[f] != synth.MASKED) & (ref["state"][0] != synth.MASKED) & (margin > 1e-3)
        mismatched_rows += int((got_tok[f][both] != ref["tokens"][0][both]).sum())
        if not amb:
            mismatched_rollouts += int(not (np.array_equal(got_st[f], ref["state"][0]) and np.array_equal(got_tok[f], ref["tokens"][0])))
        checked += 1
    return {"rollouts_checked": checked, "rows": rows, "low_margin_rows": low, "ambiguous_rollouts": ambiguous,
            "mismatched_clear_rows": mismatched_rows, "mismatched_clear_rollouts": mismatched_rollouts,
            "what": "first unmasking step of scene 0, GPU against the CPU fp64 oracle on the same inputs"}


def cpu_baseline(workload_name, budget_s=20.0):
    from paper_2605_23163_b200 import synth
    w = synth.workload(workload_name)
    cores = len(os.sched_getaffinity(0))
    try:
        from threadpoolctl import threadpool_info
        blas = [p.get("num_threads") for p in threadpool_info() if p.get("user_api") == "blas"]
        if blas:
            cores = int(max(blas))
    except Exception:
        pass
    n = w.scenes[0].n_forks
    dt = toks = steps = used = 0
    while used < n and (used == 0 or dt < 0.5 * budget_s):
        a, b, c = _oracle_block(w, used)
        dt, toks, steps, used = dt + a, toks + b, steps + c, used + 1
    return {"value": toks / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"rollouts 0..{used - 1} of {n}, one after the other: whole block loop each "
                      f"({steps} denoising steps, {toks} committed tokens in total) in {dt:.2f} s; rollouts "
                      "are independent, so tokens/s of the full workload is the same figure"}


def run_reference(args):
    rank = int(os.environ.get("RANK", 0))
    if rank != 0:
        return
    from paper_2605_23163_b200 import synth
    w = synth.workload(args.workload)
    sc = w.scenes[0]
    for i in range(args.warmup):
        _oracle_block(w, i % sc.n_forks)
    total_t, total_tok = 0.0, 0
    for i in range(args.steps):
        dt, toks, _ = _oracle_block(w, (args.warmup + i) % sc.n_forks)
        total_t += dt
        total_tok += toks
    cores = len(os.sched_getaffinity(0))
    val = total_tok / total_t
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT,
            "n_gpus": int(os.environ.get("WORLD_SIZE", 1)), "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": 1e3 * total_t / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "sample": "one rollout per step (whole block loop)"},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": "each step decodes one rollout's block with the CPU fp64 oracle"},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def spawn_ranks(n, argv):
    """`python bench.py --gpus N` without a launcher: start the N ranks (one process per GPU) through
    torch.distributed.run on this node and hand back its exit code.  Rank 0 prints the JSON line."""
    import socket
    import subprocess
    with socket.socket() as sock:                # a free port for the rendezvous
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


def run_replica_selftest(args):
    """The multi-GPU bookkeeping of the benchmark without a GPU: every rank contributes a made-up time
    and token count, rank 0 prints what run_ours would print from them (gloo on CPU)."""
    import torch.distributed as dist
    from paper_2605_23163_b200 import replicas, synth
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if world > 1:
        dist.init_process_group("gloo")
    d = dist if world > 1 else None
    w = replicas.replica_workload(synth.workload("tiny"), rank)
    ms = replicas.max_over_ranks(10.0 + rank, d)
    tokens = replicas.sum_over_ranks(12 * args.steps, d)
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": tokens / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
                          "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps,
                          "selftest": True, "seed_rank0": w.seed}))
    if world > 1:
        dist.destroy_process_group()


def main():
    global PRE_STEPS, LOOKAHEAD, COUNT_STREAM, GRAPH, NATIVE_LOOP, TIME_EVERY
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="long_prefix")
    ap.add_argument("--layers", type=int, default=1)
    ap.add_argument("--n-forks", type=int, default=0, help="override the number of rollouts of every scene")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--pre-steps", type=int, default=PRE_STEPS,
                    help="distinct per-step input sets kept resident on the device")
    ap.add_argument("--cpu-budget", type=float, default=20.0)
    ap.add_argument("--no-lookahead", action="store_true",
                    help="enqueue a denoising step only after the host has read the counts of the one before")
    ap.add_argument("--counts", choices=["auto", "in-line", "own-stream"], default="auto",
                    help="where the per-rollout counts are copied to the host: on the compute stream or on a stream of their own")
    ap.add_argument("--loop", choices=["library", "python"], default="library",
                    help="who runs the block loop of the blocks that are not timed kernel by kernel: the library's fdd_decode_block or this file")
    ap.add_argument("--time-every", type=int, default=TIME_EVERY,
                    help="every N-th block runs through the loop in this file with CUDA events around each kernel (the "
                         "per-kernel figures of the roofline objects); 0: none, every block runs as a user would run it")
    ap.add_argument("--graph", action="store_true",
                    help="replay every denoising step from a CUDA graph (blocks whose kernels are timed one by one still run call by call)")
    ap.add_argument("--selftest-replicas", action="store_true",
                    help="no GPU work: the ranks only do the replica bookkeeping (MAX of times, SUM of tokens) over gloo")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    PRE_STEPS = max(1, args.pre_steps)
    LOOKAHEAD = not args.no_lookahead
    GRAPH = args.graph
    TIME_EVERY = max(0, args.time_every)
    NATIVE_LOOP = args.loop == "library" and not args.no_lookahead
    COUNT_STREAM = {"auto": None, "in-line": False, "own-stream": True}[args.counts]
    if args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args.gpus, sys.argv[1:]))      # no launcher: start the ranks ourselves
    elif args.selftest_replicas:
        run_replica_selftest(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
