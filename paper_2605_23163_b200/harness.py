"""Device-side set-up of a synthetic scene: cache layouts, buffers, fork set.

Plumbing shared by the tests, the smoke check and the benchmark.  It moves the
arrays of `synth` into device memory in the layouts the C-ABI expects and calls
the binding; it computes nothing of the method itself and never touches the CPU
oracle.
"""
import numpy as np
import torch

from . import fdd, synth


def bf16_tensor(bits, device="cuda"):
    """uint16 bf16 bit patterns (numpy) -> torch.bfloat16 tensor on `device`."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    return t.to(device).view(torch.bfloat16)


def pack_prefix_contiguous(bits, capacity=None, device="cuda"):
    """[P, Hkv, D] bits -> bf16 [Hkv, capacity, D] (head-major contiguous cache)."""
    P, H, D = bits.shape
    capacity = capacity or max(P, 1)
    out = torch.zeros((H, capacity, D), dtype=torch.bfloat16, device=device)
    if P:
        out[:, :P] = bf16_tensor(bits, device).permute(1, 0, 2)
    return out


def pack_prefix_paged(bits, page_tokens, page_ids, pool_pages, device="cuda"):
    """[P, Hkv, D] bits -> bf16 [pool_pages, Hkv, page_tokens, D]; logical page j lives in
    physical page page_ids[j].  Unused slots are zero."""
    P, H, D = bits.shape
    n_pages = (P + page_tokens - 1) // page_tokens
    padded = np.zeros((n_pages * page_tokens, H, D), dtype=np.uint16)
    padded[:P] = bits
    src = bf16_tensor(padded, device).view(n_pages, page_tokens, H, D).permute(0, 2, 1, 3)
    out = torch.zeros((pool_pages, H, page_tokens, D), dtype=torch.bfloat16, device=device)
    out[torch.as_tensor(np.asarray(page_ids[:n_pages]), device=device, dtype=torch.long)] = src
    return out


class GpuScene:
    """One scene of a workload resident on the GPU: shared prefix cache (per layer),
    private suffix buffers and the fork set made from them."""

    def __init__(self, ctx, w, scene_idx, n_layers=1, suffix_capacity=None, device="cuda",
                 identical_seeds=False, distinct_layer_caches=True):
        self.ctx, self.w, self.scene_idx = ctx, w, scene_idx
        sc = w.scenes[scene_idx]
        self.sc = sc
        self.n_layers = n_layers
        self.suffix_capacity = suffix_capacity or sc.block_len * max(sc.n_blocks, 1)
        self.prefix_k, self.prefix_v = [], []
        self.page_table = None
        pt = w.page_tokens
        if pt:
            n_pages = (sc.prefix_len + pt - 1) // pt
            self.pool_pages = n_pages + 3
            ids = synth.page_order(w, scene_idx, n_pages, self.pool_pages)
            self.page_table = torch.from_numpy(ids).to(device)
            self.prefix_capacity = self.pool_pages
        else:
            self.prefix_capacity = max(sc.prefix_len, 1)
        for layer in range(n_layers):
            src = layer if distinct_layer_caches else 0
            kb, vb = synth.make_prefix(w, scene_idx, src)
            if pt:
                self.prefix_k.append(pack_prefix_paged(kb, pt, ids, self.pool_pages, device))
                self.prefix_v.append(pack_prefix_paged(vb, pt, ids, self.pool_pages, device))
            else:
                self.prefix_k.append(pack_prefix_contiguous(kb, self.prefix_capacity, device))
                self.prefix_v.append(pack_prefix_contiguous(vb, self.prefix_capacity, device))
        shape = (sc.n_forks, w.n_kv_heads, self.suffix_capacity, w.head_dim)
        self.suffix_k = [torch.zeros(shape, dtype=torch.bfloat16, device=device) for _ in range(n_layers)]
        self.suffix_v = [torch.zeros(shape, dtype=torch.bfloat16, device=device) for _ in range(n_layers)]
        self.seeds = synth.fork_seeds(w, scene_idx, identical=identical_seeds)
        self.forkset = fdd.fdd_fork(ctx, self.prefix_k, self.prefix_v, self.page_table, sc.prefix_len,
                                    self.prefix_capacity, sc.n_forks, self.seeds,
                                    self.suffix_k, self.suffix_v, self.suffix_capacity)

    def free(self):
        if self.forkset is not None:
            fdd.fdd_forkset_free(self.ctx, self.forkset)
            self.forkset = None


def create_context(w, n_layers=1, max_forks=None, max_block=None):
    """An fdd context sized for workload `w`."""
    total_forks = max_forks or sum(s.n_forks for s in w.scenes)
    blk = max_block or max(s.block_len for s in w.scenes)
    return fdd.fdd_create(w.n_q_heads, w.n_kv_heads, w.head_dim, w.vocab, n_layers, w.page_tokens,
                          blk, total_forks,
                          fdd.FDD_LOGITS_BF16 if w.logits_dtype == "bf16" else fdd.FDD_LOGITS_F32)


def logits_tensor(w, arr, device="cuda"):
    """numpy logits (fp32 values or bf16 bits) -> device tensor of the configured dtype."""
    if w.logits_dtype == "bf16":
        return bf16_tensor(arr, device)
    return torch.from_numpy(np.ascontiguousarray(arr)).to(device)
