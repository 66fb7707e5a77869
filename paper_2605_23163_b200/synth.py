"""Seeded synthetic inputs shaped like the paper's driving workloads.

This module only *makes inputs*: random tensors with the shapes, value
distributions and structure of the decode workloads (a long multi-camera
visual+text prefix, short JSON-section blocks with a fixed share of frozen
scaffold positions, N rollouts).  It contains none of the decode arithmetic
(no attention, no unmasking rule, no noise generator) and imports neither the
CUDA binding nor the CPU oracle; both sides of a parity test feed on the same
arrays produced here.  The driving datasets, the tokenizer and the trained
weights are not available, so these arrays stand in for them.

Every array is a pure function of (workload seed, scene, layer, block, step,
tensor name[, rollout, position]), so any single row can be regenerated
without materialising the rest.

bfloat16 tensors are returned as uint16 bit patterns (round-to-nearest-even
from fp32, done once here) so that every consumer sees identical bits.
"""
from dataclasses import dataclass, field
import numpy as np

MASKED, COMMITTED, SCAFFOLD = 0, 1, 2

_NAMES = {"prefix_k": 1, "prefix_v": 2, "q": 3, "k": 4, "v": 5, "logits": 6,
          "scaffold": 7, "tokens": 8, "scene": 9, "traj": 10, "pages": 11}


@dataclass(frozen=True)
class Scene:
    prefix_len: int
    n_forks: int
    block_len: int
    n_scaffold: int          # frozen positions per block
    n_blocks: int = 1


@dataclass(frozen=True)
class Workload:
    name: str
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    vocab: int
    logits_dtype: str        # "f32" or "bf16"
    logit_recipe: str        # "normal_sigma2", "peaked" or "constant"
    threshold: float
    temperature: float
    scenes: tuple
    qkv_sigma: float = 1.0
    page_tokens: int = 0     # 0 = contiguous prefix cache
    n_layers: int = 1
    seed: int = 0
    waypoints: int = 10
    notes: str = ""

    @property
    def group(self):
        return self.n_q_heads // self.n_kv_heads

    @property
    def mask_id(self):
        return self.vocab - 1


def _c5_scenes(seed=5):
    g = np.random.default_rng(np.random.SeedSequence(entropy=seed, spawn_key=(_NAMES["scene"],)))
    scenes = []
    for _ in range(16):
        p = int(g.integers(2048, 12289))
        n = int(g.choice([1, 4, 16]))
        d = int(g.choice([16, 32, 64]))
        scenes.append(Scene(prefix_len=p, n_forks=n, block_len=d, n_scaffold=int(round(0.3 * d))))
    return tuple(scenes)


def workload(name):
    """The five benchmark configurations, by name ("tiny", "single_scene",
    "tts", "long_prefix", "serving_mix")."""
    if name == "tiny":
        return Workload("tiny", 4, 1, 64, 4096, "f32", "normal_sigma2", 0.9, 0.0,
                        (Scene(256, 1, 16, 4, 1),), qkv_sigma=1.0 / 8.0, seed=0)
    if name == "single_scene":
        return Workload("single_scene", 16, 2, 128, 151936, "bf16", "peaked", 0.9, 0.0,
                        (Scene(4096, 1, 32, 10, 6),), seed=2)
    if name == "tts":
        return Workload("tts", 16, 2, 128, 151936, "bf16", "peaked", 0.9, 1.0,
                        (Scene(4096, 8, 32, 10, 6),), seed=3)
    if name == "long_prefix":
        return Workload("long_prefix", 32, 8, 128, 151936, "bf16", "peaked", 0.8, 1.0,
                        (Scene(16384, 32, 64, 26, 1),), seed=4)
    if name == "serving_mix":
        return Workload("serving_mix", 16, 2, 128, 151936, "bf16", "peaked", 0.9, 1.0,
                        _c5_scenes(), page_tokens=64, seed=5)
    raise KeyError(name)


WORKLOADS = ("tiny", "single_scene", "tts", "long_prefix", "serving_mix")


def small_variant(w, prefix_len=None, vocab=None, n_forks=None, n_blocks=None, name=None):
    """A reduced copy of a workload (same head geometry and recipe) for parity
    cases the oracle can finish quickly."""
    scenes = tuple(Scene(prefix_len or s.prefix_len, n_forks or s.n_forks, s.block_len,
                         s.n_scaffold, n_blocks or s.n_blocks) for s in w.scenes)
    return Workload(name or (w.name + "_small"), w.n_q_heads, w.n_kv_heads, w.head_dim,
                    vocab or w.vocab, w.logits_dtype, w.logit_recipe, w.threshold,
                    w.temperature, scenes, w.qkv_sigma, w.page_tokens, w.n_layers, w.seed,
                    w.waypoints, w.notes)


# ----------------------------------------------------------------------------
# bf16 bit helpers (input formatting only)
# ----------------------------------------------------------------------------
def f32_to_bf16_bits(x):
    """Round fp32 to bfloat16 (nearest even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits):
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(w, name, *key):
    return np.random.default_rng(np.random.SeedSequence(
        entropy=int(w.seed), spawn_key=(_NAMES[name],) + tuple(int(k) for k in key)))


# ----------------------------------------------------------------------------
# tensors
# ----------------------------------------------------------------------------
def make_prefix(w, scene_idx, layer=0):
    """Shared prefix K and V, logical layout [P, Hkv, D], bf16 bits."""
    sc = w.scenes[scene_idx]
    shape = (sc.prefix_len, w.n_kv_heads, w.head_dim)
    k = _rng(w, "prefix_k", scene_idx, layer).standard_normal(shape, dtype=np.float32) * np.float32(w.qkv_sigma)
    v = _rng(w, "prefix_v", scene_idx, layer).standard_normal(shape, dtype=np.float32) * np.float32(w.qkv_sigma)
    return f32_to_bf16_bits(k), f32_to_bf16_bits(v)


def make_qkv(w, scene_idx, layer, block, step):
    """Projections of the current block for one denoising step:
    q [N, d, Hq, D], k, v [N, d, Hkv, D], bf16 bits."""
    sc = w.scenes[scene_idx]
    out = []
    for name, heads in (("q", w.n_q_heads), ("k", w.n_kv_heads), ("v", w.n_kv_heads)):
        shape = (sc.n_forks, sc.block_len, heads, w.head_dim)
        x = _rng(w, name, scene_idx, layer, block, step).standard_normal(shape, dtype=np.float32)
        out.append(f32_to_bf16_bits(x * np.float32(w.qkv_sigma)))
    return tuple(out)


def scaffold_positions(w, scene_idx, block):
    """Sorted indices of the frozen positions of a block (fixed, seeded)."""
    sc = w.scenes[scene_idx]
    g = _rng(w, "scaffold", scene_idx, block)
    return np.sort(g.choice(sc.block_len, size=sc.n_scaffold, replace=False))


def make_block_template(w, scene_idx, block):
    """tokens [N, d] int32 and state [N, d] uint8 at the start of a block:
    scaffold positions pre-filled and SCAFFOLD, value positions mask_id and
    MASKED; identical for every rollout."""
    sc = w.scenes[scene_idx]
    pos = scaffold_positions(w, scene_idx, block)
    tok = np.full(sc.block_len, w.mask_id, dtype=np.int32)
    st = np.full(sc.block_len, MASKED, dtype=np.uint8)
    tok[pos] = _rng(w, "tokens", scene_idx, block).integers(0, w.vocab - 1, size=len(pos), dtype=np.int32)
    st[pos] = SCAFFOLD
    return (np.tile(tok, (sc.n_forks, 1)), np.tile(st, (sc.n_forks, 1)))


def make_logits_row(w, scene_idx, block, step, fork, pos):
    """One row of vocabulary logits.

    "normal_sigma2": iid N(0, sigma = 2) in fp32 (never confident: exercises
    the at-least-one rule).  "peaked": iid N(0, 1) with one seeded entry raised
    to logsumexp(rest) + m, m ~ U(0, 6), so the soft-max maximum is sigmoid(m)
    in [0.5, 0.9975] and a threshold of 0.8-0.9 is reached by most rows.
    "constant": every entry of the row has the same seeded value (the degenerate
    case in which sampling noise alone decides the token).
    Returns fp32 values ("f32") or bf16 bits ("bf16").
    """
    g = _rng(w, "logits", scene_idx, block, step, fork, pos)
    if w.logit_recipe == "normal_sigma2":
        row = g.standard_normal(w.vocab, dtype=np.float32) * np.float32(2.0)
    elif w.logit_recipe == "peaked":
        row = g.standard_normal(w.vocab, dtype=np.float32)
        if w.logits_dtype == "bf16":
            row = bf16_bits_to_f32(f32_to_bf16_bits(row))
        t = int(g.integers(0, w.vocab))
        m = float(g.uniform(0.0, 6.0))
        r64 = row.astype(np.float64)
        r64[t] = -np.inf
        mx = float(np.max(r64))
        lse = mx + float(np.log(np.sum(np.exp(r64 - mx))))
        row[t] = np.float32(lse + m)
    elif w.logit_recipe == "constant":
        row = np.full(w.vocab, np.float32(g.uniform(-3.0, 3.0)), dtype=np.float32)
    else:
        raise ValueError(w.logit_recipe)
    if w.logits_dtype == "bf16":
        return f32_to_bf16_bits(row)
    return row


def make_logits(w, scene_idx, block, step, rows="value"):
    """Logits [N, d, V] for one step.  rows="value": only non-scaffold rows are
    generated (scaffold rows are never read by the method and stay zero);
    rows="all": every row."""
    sc = w.scenes[scene_idx]
    dt = np.uint16 if w.logits_dtype == "bf16" else np.float32
    out = np.zeros((sc.n_forks, sc.block_len, w.vocab), dtype=dt)
    frozen = set(scaffold_positions(w, scene_idx, block).tolist()) if rows == "value" else set()
    for f in range(sc.n_forks):
        for i in range(sc.block_len):
            if i not in frozen:
                out[f, i] = make_logits_row(w, scene_idx, block, step, f, i)
    return out


def fork_seeds(w, scene_idx, identical=False):
    """64-bit seeds per rollout: base + f (or all equal for the identity test)."""
    sc = w.scenes[scene_idx]
    base = np.uint64((0x9E3779B97F4A7C15 * (w.seed * 1000 + scene_idx + 1)) & 0xFFFFFFFFFFFFFFFF)
    f = np.zeros(sc.n_forks, dtype=np.uint64) if identical else np.arange(sc.n_forks, dtype=np.uint64)
    return base + f


def page_order(w, scene_idx, n_pages, pool_pages):
    """A seeded, shuffled choice of physical pages for a paged prefix."""
    g = _rng(w, "pages", scene_idx)
    return g.permutation(pool_pages)[:n_pages].astype(np.int32)


def tokens_to_trajectory(w, tokens, state):
    """Synthetic stand-in for reading a trajectory out of decoded tokens (the
    tokenizer is unavailable): the value tokens of each rollout, in order, six
    per coordinate (sign = (id // 10) % 2, digit = id % 10, format +-ddd.dd);
    missing digits count as zero.  tokens/state: [N, T].  Returns [N, W, 2]
    fp32."""
    tokens = np.asarray(tokens)
    state = np.asarray(state)
    n = tokens.shape[0]
    out = np.zeros((n, w.waypoints, 2), dtype=np.float32)
    need = w.waypoints * 2 * 6
    for f in range(n):
        vals = tokens[f][state[f] != SCAFFOLD].astype(np.int64)[:need]
        vals = np.concatenate([vals, np.zeros(need - len(vals), dtype=np.int64)])
        vals = vals.reshape(w.waypoints, 2, 6)
        sign = np.where((vals[..., 0] // 10) % 2 == 0, 1.0, -1.0)
        digits = vals[..., 1:] % 10
        mag = (digits * np.array([100.0, 10.0, 1.0, 0.1, 0.01])).sum(-1)
        out[f] = (sign * mag).astype(np.float32)
    return out
